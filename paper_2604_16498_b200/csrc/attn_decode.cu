// Split-KV decode attention and its combine step: Eq. 9 for a single query row per head
// over the first lens[b] rows of a KV cache.  The cached sequence is cut into num_splits
// ranges; each range yields a partial (running max m, running sum l, unnormalised output)
// and the combine step merges the partials:
//     M = max_s m_s,   L = sum_s 2^(m_s - M) l_s,   out = sum_s 2^(m_s - M) O_s / L
// (scores are kept in log2 units: they are multiplied by scale * log2(e)).
//
// The work is bound by streaming K and V from HBM once, and HBM only delivers its bandwidth
// with a deep queue of requests (pure streaming with 48 KB in flight per SM reaches 4.2 TB/s on
// this part, with 250 KB 5.8 TB/s).  So the split kernel is persistent and every warp is an
// independent worker: it owns whole (batch, kv head, split) items, keeps a private ring of
// 16-row blocks in shared memory filled by TMA tile copies (16 rows x 64 columns each, 128-byte
// swizzle, completion counted on an mbarrier per stage) that run ahead across item boundaries
// (8 warps x 24 KB in flight per SM), and writes its partial straight from registers.  Split
// boundaries are multiples of 16 rows, so a block never straddles two splits.  No warp ever waits for another one.  Items differ in length by up to the ratio of the
// longest to the shortest cached sequence, so they are dealt out longest sequence first and in
// alternating direction from round to round (a worker that got one of the longest items in one round
// gets one of the shortest in the next), which keeps the workers' totals close together.
// The G = Hq / Hkv query heads that share a KV
// head are processed together, so every cached row is read exactly once.  The dot products run
// on warp-level tensor-core MMAs (m16n8k16) with fragments read from the swizzled ring; fp32 FMAs
// with shuffle reductions were bound by instruction issue.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <mutex>

#include "forge_common.cuh"
#include "sm100_ptx.cuh"
#include "tmap.cuh"

namespace forge {
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kBlockKeys = 16;             // cached rows per ring stage
constexpr int kWarpRingBytes = 24 * 1024;  // per warp
constexpr int kMaxSortedBatch = 64;        // batches up to this size are ordered by cached length

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col).  Lane = (g = lane / 4, c = lane % 4):
//   A: a0 = (row g, k 2c..2c+1)  a1 = (row g+8, k 2c..)  a2 = (row g, k 2c+8..)  a3 = (row g+8, k 2c+8..)
//   B: b0 = (k 2c..2c+1, col g)  b1 = (k 2c+8.., col g)
//   D: d0 = (row g, col 2c)  d1 = (row g, col 2c+1)  d2 = (row g+8, col 2c)  d3 = (row g+8, col 2c+1)
// F16 selects fp16 operands instead of bf16 (the same fragment layout).
template <bool F16>
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    if constexpr (F16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
                     "{%8, %9}, {%0, %1, %2, %3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
                     "{%8, %9}, {%0, %1, %2, %3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <bool F16>
__device__ __forceinline__ uint32_t pack16x2(float lo, float hi) {
    if constexpr (F16) {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    } else {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
}

// One (batch, kv head, split) work item and its range of cached rows.
struct Item {
    int b, kvh, split, s0, s1;
};
// idx counts items in dealing order: all (kv head, split) pairs of the longest sequence, then of the
// next one, ...; order[r] is the batch entry with the r-th longest cached sequence (nullptr: identity).
__device__ __forceinline__ Item make_item(int idx, const int32_t* lens, const int* order, int Hkv, int Smax,
                                          int num_splits) {
    Item it;
    it.split = idx % num_splits;
    const int bk = idx / num_splits;
    it.kvh = bk % Hkv;
    it.b = bk / Hkv;
    if (order) it.b = order[it.b];
    const int len = min(max(lens[it.b], 0), Smax);
    // rows per split: the even share, rounded up to whole 16-row blocks
    const int per = (((len + num_splits - 1) / num_splits) + kBlockKeys - 1) / kBlockKeys * kBlockKeys;
    it.s0 = it.split * per;
    it.s1 = min(it.s0 + per, len);
    if (it.s1 < it.s0) it.s1 = it.s0;
    return it;
}

// Worker w (= warp) takes items w, w + workers, ...; consecutive items go to different SMs.
//   S[head, key]  = Q K^T   as m16n8k16 with A = Q (rows = the G heads, padded with zero rows) and
//                   B = K rows (the contraction runs over the head dimension in whatever order the
//                   16-byte chunks deliver it, the same for Q and K);
//   online softmax on the accumulator fragment (lane (g, c) owns head g, keys 2c, 2c+1 of each 8);
//   O^T[dim, head] += V^T P^T  with A = pairs of V rows interleaved with byte permutes and B = the
//                   probabilities exactly where the first MMA left them.
template <int D, int G, bool F16>
__global__ void __launch_bounds__(kThreads, 1)
decode_split_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                    const uint16_t* __restrict__ q, const int32_t* __restrict__ lens,
                    float* __restrict__ ws_o, float* __restrict__ ws_ml,
                    int B, int Hq, int Hkv, int Smax, int head_dim, int num_splits, float scale_log2, int* status) {
    constexpr int NKB = D / 32;  // 32-dim blocks of the head dimension (two k16 MMAs each)
    constexpr int NHB = D / 64;  // 64-dim blocks of the output (four 16-dim MMAs each)
    // A stage holds 16 rows of K and 16 rows of V as D / 64 tiles of 16 rows x 128 bytes each; 16-byte chunk
    // k of row r of a tile sits at r * 128 + ((k ^ (r & 7)) << 4) (the TMA unit's 128-byte swizzle).
    constexpr int kTileBytes = kBlockKeys * 128;
    constexpr int kKBytes = (D / 64) * kTileBytes;
    constexpr int kStageBytes = 2 * kKBytes;
    constexpr int kStages = kWarpRingBytes / kStageBytes;  // 3 for D = 128, 6 for D = 64
    static_assert(kStages >= 2 && kStages <= 8, "ring size");

    // Let the combine kernel (launched with programmatic stream serialisation) become resident right
    // away: its CTAs are small, sit next to this one and block in griddepcontrol.wait until this grid
    // has completed and its writes are visible, so the merge starts without a launch gap.
    pdl_launch_dependents();
    pdl_wait();  // the previous kernel in the stream has completed (this kernel may have been resident before)
    extern __shared__ __align__(128) uint8_t ring_raw[];
    __shared__ uint64_t full_bars[kWarps][8];  // [warp][stage]: the stage's rows have landed
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, c = lane & 3;
    // swizzled tiles need 1024-byte alignment
    const uint32_t ring = ((static_cast<uint32_t>(__cvta_generic_to_shared(ring_raw)) + 1023u) & ~1023u) +
                          warp * kWarpRingBytes;
    uint64_t* full = full_bars[warp];
    if (lane == 0) {
        for (int i = 0; i < kStages; ++i) ptx::mbar_init(&full[i], 1);
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_k);
        ptx::prefetch_tmap(&tmap_v);
    }
    __syncwarp();

    const int num_items = B * Hkv * num_splits;
    const int workers = gridDim.x * kWarps;
    const int worker = warp * gridDim.x + blockIdx.x;

    // ---- dealing order of the batch entries: longest cached sequence first (ties by index)
    __shared__ int order_smem[kMaxSortedBatch];
    const int* order = nullptr;
    if (B <= kMaxSortedBatch) {
        if (tid < B) {
            const int mine = min(max(lens[tid], 0), Smax);
            int rank = 0;
            for (int o = 0; o < B; ++o) {
                const int other = min(max(lens[o], 0), Smax);
                rank += (other > mine) || (other == mine && o < tid);
            }
            order_smem[rank] = tid;
        }
        __syncthreads();
        order = order_smem;
    }
    // the item of this worker in round r: rounds alternate in direction
    auto item_of_round = [&](int r) { return r * workers + ((r & 1) ? workers - 1 - worker : worker); };

    // ---- prefetch cursor: runs kStages blocks ahead of the compute, across item boundaries (a stage is
    // refilled as soon as its fragments are in registers, before the MMAs on them)
    int p_round = 0, p_idx = item_of_round(0), p_j0 = 0, p_s1 = 0;
    int p_bk = 0;  // batch * Hkv + kv head of the cursor's item
    int p_n = 0;  // blocks issued
    auto p_open = [&]() {  // position the cursor on the first block of the next non-empty item
        while (p_idx < num_items) {
            const Item it = make_item(p_idx, lens, order, Hkv, Smax, num_splits);
            if (it.s1 > it.s0) {
                p_j0 = it.s0;
                p_s1 = it.s1;
                p_bk = it.b * Hkv + it.kvh;
                return;
            }
            p_idx = item_of_round(++p_round);
        }
    };
    auto issue = [&]() {  // one lane starts the block's tile copies (rows past the cache's end are zero-filled)
        if (p_idx < num_items) {
            if (lane == 0) {
                const int st = p_n % kStages;
                const uint32_t dst = ring + st * kStageBytes;
                ptx::mbar_expect_tx(&full[st], kStageBytes);
#pragma unroll
                for (int cb = 0; cb < D / 64; ++cb) {
                    ptx::tma_load_3d_addr(dst + cb * kTileBytes, &tmap_k, &full[st], cb * 64, p_j0, p_bk);
                    ptx::tma_load_3d_addr(dst + kKBytes + cb * kTileBytes, &tmap_v, &full[st], cb * 64, p_j0, p_bk);
                }
            }
            ++p_n;
            p_j0 += kBlockKeys;
            if (p_j0 >= p_s1) { p_idx = item_of_round(++p_round); p_open(); }
        }
    };
    p_open();
#pragma unroll
    for (int i = 0; i < kStages; ++i) issue();

    // Q fragment of an item: head g (zero rows for g >= G), 8 dims at c*8 of every 32-dim block
    auto load_q = [&](const Item& it, uint32_t (&qr)[NKB][4]) {
#pragma unroll
        for (int kb = 0; kb < NKB; ++kb) {
            uint4 raw = make_uint4(0, 0, 0, 0);
            if (g < G && kb * 32 + c * 8 < head_dim)  // dims beyond the tensors' head size count as zeros
                raw = *reinterpret_cast<const uint4*>(q + ((size_t)it.b * Hq + it.kvh * G + g) * head_dim + kb * 32 + c * 8);
            qr[kb][0] = raw.x; qr[kb][1] = raw.y; qr[kb][2] = raw.z; qr[kb][3] = raw.w;
        }
    };

    Item nxt = {0, 0, 0, 0, 0};
    uint32_t qn[NKB][4];
    if (item_of_round(0) < num_items) {
        nxt = make_item(item_of_round(0), lens, order, Hkv, Smax, num_splits);
        load_q(nxt, qn);
    }
    int n = 0;  // blocks consumed
    bool failed = false;
    for (int round = 0; item_of_round(round) < num_items; ++round) {
        const Item it = nxt;
        uint32_t qr[NKB][4];
#pragma unroll
        for (int kb = 0; kb < NKB; ++kb)
#pragma unroll
            for (int i = 0; i < 4; ++i) qr[kb][i] = qn[kb][i];
        if (item_of_round(round + 1) < num_items) {  // fetch the next item's range and Q rows early
            nxt = make_item(item_of_round(round + 1), lens, order, Hkv, Smax, num_splits);
            load_q(nxt, qn);
        }

        float m_run = -INFINITY, l_run = 0.f;  // of head g (lanes with g >= G carry dummies)
        float acc[NHB][4][4];                  // O^T fragments: [64-dim block][16-dim MMA][d0..d3]
#pragma unroll
        for (int hb = 0; hb < NHB; ++hb)
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[hb][t][i] = 0.f;

        for (int j0 = it.s0; j0 < it.s1; j0 += kBlockKeys, ++n) {
            // the rows of block n have landed (bounded wait: on expiry the kernel flags the error and leaves)
            if (!ptx::warp_wait(&full[n % kStages], (n / kStages) & 1)) { failed = true; break; }
            const uint32_t sa = ring + (n % kStages) * kStageBytes;
            // K fragment: rows u*8 + g, chunk kb*4 + c.  V fragment: rows {2c, 2c+1, 2c+8, 2c+9}, chunk hb*8 + g.
            uint4 kr[2][NKB], vr[4][NHB];
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int kb = 0; kb < NKB; ++kb)
                    kr[u][kb] = lds128(sa + (kb / 2) * kTileBytes + (u * 8 + g) * 128 + ((((kb & 1) * 4 + c) ^ g) << 4));
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int row = 2 * c + (r & 1) + (r >> 1) * 8;
#pragma unroll
                for (int hb = 0; hb < NHB; ++hb)
                    vr[r][hb] = lds128(sa + kKBytes + hb * kTileBytes + row * 128 + ((g ^ (row & 7)) << 4));
                // a row past the sequence's end holds whatever the cache holds there: it must not reach the MMA
                // (its probability is 0, but 0 x NaN is NaN)
                if (j0 + row >= it.s1) {
#pragma unroll
                    for (int hb = 0; hb < NHB; ++hb) vr[r][hb] = make_uint4(0, 0, 0, 0);
                }
            }
            __syncwarp();  // all fragment reads done before this stage is refilled ...
            ptx::fence_proxy_async_smem();  // ... by the copy engine (reads before its writes)
            issue();

            // scores: s[u][0..1] = head g, keys j0 + u*8 + 2c + {0, 1}  (s[u][2..3] belong to zero rows)
            float s[2][4];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                // two accumulation chains per key group (shorter dependent MMA sequences)
                float s2[4] = {0.f, 0.f, 0.f, 0.f};
                s[u][0] = s[u][1] = s[u][2] = s[u][3] = 0.f;
#pragma unroll
                for (int kb = 0; kb < NKB; ++kb) {
                    mma16816<F16>(s[u], qr[kb][0], 0u, qr[kb][1], 0u, kr[u][kb].x, kr[u][kb].y);
                    mma16816<F16>(s2, qr[kb][2], 0u, qr[kb][3], 0u, kr[u][kb].z, kr[u][kb].w);
                }
                s[u][0] += s2[0];
                s[u][1] += s2[1];
            }
            float mt = -INFINITY;
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const bool ok = (j0 + u * 8 + 2 * c + i) < it.s1;
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

            // P^T as the B operand: k-slots (2c, 2c+1) = keys 2c, 2c+1; (2c+8, 2c+9) = keys 2c+8, 2c+9
            const uint32_t pb0 = pack16x2<F16>(p[0][0], p[0][1]);
            const uint32_t pb1 = pack16x2<F16>(p[1][0], p[1][1]);
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
                for (int t = 0; t < 4; ++t) mma16816<F16>(acc[hb][t], ab[t], ab[4 + t], cd[t], cd[4 + t], pb0, pb1);
            }
        }

        if (failed) break;
        // ---- this warp's partial is the item's partial: write it out from the fragments
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        const size_t slot0 = ((size_t)it.b * Hq + it.kvh * G) * num_splits + it.split;  // head 0 of the group
        if (g < G && c == 0) {
            ws_ml[(slot0 + (size_t)g * num_splits) * 2] = m_run;
            ws_ml[(slot0 + (size_t)g * num_splits) * 2 + 1] = l_run;
        }
        if (it.s1 > it.s0) {  // an empty split has m = -inf and its output slot is never read
#pragma unroll
            for (int hb = 0; hb < NHB; ++hb)
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int d0 = hb * 64 + g * 8 + t;
                    if (2 * c < G) {
                        float* o = ws_o + (slot0 + (size_t)(2 * c) * num_splits) * D;
                        o[d0] = acc[hb][t][0];
                        o[d0 + 4] = acc[hb][t][2];
                    }
                    if (2 * c + 1 < G) {
                        float* o = ws_o + (slot0 + (size_t)(2 * c + 1) * num_splits) * D;
                        o[d0] = acc[hb][t][1];
                        o[d0 + 4] = acc[hb][t][3];
                    }
                }
        }
    }
    if (failed) {
        if (lane == 0) atomicExch(status, 1);
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies in flight land before the ring goes away
    }
}

// grid = B * Hq, block = D threads: merges the num_splits partials of one (batch, head).  The
// partials are read in groups of 16 with all loads of a group in flight together.
template <int D, bool F16>
__global__ void __launch_bounds__(D)
decode_combine_kernel(const float* __restrict__ ws_o, const float* __restrict__ ws_ml,
                      uint16_t* __restrict__ out, int num_splits, int head_dim) {
    const size_t bh = blockIdx.x;
    const int d = threadIdx.x;
    const float2* ml = reinterpret_cast<const float2*>(ws_ml) + bh * num_splits;
    const float* po = ws_o + bh * num_splits * D + d;
    pdl_launch_dependents();  // the next kernel in the stream may move in while this one runs
    // the split kernel's writes are visible only after this returns
    pdl_wait();
    float M = -INFINITY, L = 0.f, O = 0.f;  // running merge over the groups
    for (int s0 = 0; s0 < num_splits; s0 += 16) {
        float2 mls[16];
        float os[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const bool ok = s0 + i < num_splits;
            mls[i] = ok ? ml[s0 + i] : make_float2(-INFINITY, 0.f);
            // the output slot of an empty split (m = -inf) was never written: whatever is read gets weight 0
            // through the select below
            os[i] = ok ? po[(size_t)(s0 + i) * D] : 0.f;
        }
        float Mg = M;
#pragma unroll
        for (int i = 0; i < 16; ++i) Mg = fmaxf(Mg, mls[i].x);
        if (Mg == -INFINITY) continue;
        const float keep = exp2f(M - Mg);  // 0 while nothing has been merged yet
        L *= keep;
        O *= keep;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float wgt = exp2f(mls[i].x - Mg);
            L = fmaf(wgt, mls[i].y, L);
            O = fmaf(wgt, (mls[i].x == -INFINITY) ? 0.f : os[i], O);
        }
        M = Mg;
    }
    const float res = L > 0.f ? O / L : 0.f;
    if (d >= head_dim) return;  // padding columns of a head size below the kernel's
    if constexpr (F16) out[bh * head_dim + d] = __half_as_ushort(__float2half_rn(res));
    else out[bh * head_dim + d] = __bfloat16_as_ushort(__float2bfloat16_rn(res));
}

template <int D, int G, bool F16>
int launch_split(const void* q, const void* kc, const void* vc, const int32_t* lens, float* ws_o, float* ws_ml,
                 int B, int Hq, int Hkv, int Smax, int head_dim, int num_splits, float scale_log2, cudaStream_t s) {
    constexpr int kSmem = kWarps * kWarpRingBytes + 1024;
    int* status = device_status_word();
    if (!status) return FORGE_ERR_CUDA;
    CUtensorMap tk, tv;
    {
        const uint32_t box[3] = {64, (uint32_t)kBlockKeys, 1};
        // rows of head_dim <= D elements: the TMA unit zero-fills the columns up to D
        const uint64_t dims[3] = {(uint64_t)head_dim, (uint64_t)Smax, (uint64_t)B * Hkv};
        const uint64_t strides[2] = {(uint64_t)head_dim * 2, (uint64_t)Smax * head_dim * 2};
        if (!encode_tmap_bf16_sw128(&tk, kc, 3, dims, strides, box)) return FORGE_ERR_CUDA;
        if (!encode_tmap_bf16_sw128(&tv, vc, 3, dims, strides, box)) return FORGE_ERR_CUDA;
    }
    auto kernel = decode_split_kernel<D, G, F16>;
    FORGE_SET_SMEM_ONCE(kernel, kSmem);
    const int sms = sm_count();
    if (sms <= 0) return FORGE_ERR_CUDA;
    const long long items = (long long)B * Hkv * num_splits;
    const long long ctas = (items + kWarps - 1) / kWarps;
    const int grid = ctas < sms ? (int)ctas : sms;
    FORGE_CUDA_TRY(launch_pdl(kernel, dim3(grid), dim3(kThreads), kSmem, s, tk, tv, static_cast<const uint16_t*>(q),
                              lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, status));
    return FORGE_OK;
}

template <int D, bool F16>
int dispatch_g(int G, const void* q, const void* kc, const void* vc, const int32_t* lens, float* ws_o,
               float* ws_ml, int B, int Hq, int Hkv, int Smax, int head_dim, int num_splits, float scale_log2,
               cudaStream_t s) {
    switch (G) {
        case 1: return launch_split<D, 1, F16>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, s);
        case 2: return launch_split<D, 2, F16>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, s);
        case 3: return launch_split<D, 3, F16>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, s);
        case 4: return launch_split<D, 4, F16>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, s);
        case 5: return launch_split<D, 5, F16>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, s);
        case 6: return launch_split<D, 6, F16>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, s);
        case 7: return launch_split<D, 7, F16>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, s);
        case 8: return launch_split<D, 8, F16>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, num_splits, scale_log2, s);
        default: return FORGE_ERR_UNSUPPORTED;
    }
}

}  // namespace
}  // namespace forge

extern "C" size_t forge_attn_decode_workspace_bytes(int B, int Hq, int D, int num_splits) {
    if (B <= 0 || Hq <= 0 || D <= 0 || num_splits <= 0) return 0;
    const size_t slots = (size_t)B * Hq * num_splits;
    const int dp = D <= 64 ? 64 : 128;  // the partial outputs are as wide as the kernel's head dimension
    return (slots * (size_t)(dp + 2) * sizeof(float) + 15) & ~(size_t)15;
}

namespace forge {
namespace {

template <bool F16>
int decode_splitkv_impl(const void* q, const void* k_cache, const void* v_cache, void* out,
                        int B, int Hq, int Hkv, int Smax, int D,
                        const int32_t* lens, int num_splits, float scale,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if (!lens) return FORGE_ERR_INVALID_ARG;
    int st = check_attn_args(q, k_cache, v_cache, out, B, Hq, Hkv, 1, Smax, D, FORGE_MASK_PADDING, lens, /*any_head_dim=*/true);
    if (st != FORGE_OK) return st;
    if (num_splits < 1) return FORGE_ERR_INVALID_ARG;
    if (num_splits > 64 || Hkv > 65535 || B > 65535) return FORGE_ERR_UNSUPPORTED;
    if (!workspace || !aligned16(workspace)) return FORGE_ERR_INVALID_ARG;
    if (workspace_bytes < forge_attn_decode_workspace_bytes(B, Hq, D, num_splits)) return FORGE_ERR_WORKSPACE;

    const size_t slots = (size_t)B * Hq * num_splits;
    float* ws_o = static_cast<float*>(workspace);
    float* ws_ml = ws_o + slots * (D <= 64 ? 64 : 128);
    const float scale_log2 = scale * 1.4426950408889634f;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int G = Hq / Hkv;
    st = (D <= 64) ? dispatch_g<64, F16>(G, q, k_cache, v_cache, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, D, num_splits, scale_log2, s)
                   : dispatch_g<128, F16>(G, q, k_cache, v_cache, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, D, num_splits, scale_log2, s);
    if (st != FORGE_OK) return st;
    st = finish_launch(1);
    if (st != FORGE_OK) return st;
    // The combine kernel is launched with programmatic stream serialisation: its CTAs may be placed
    // while the split kernel drains, and block in griddepcontrol.wait until that grid has completed.
    const float* cws_o = ws_o;
    const float* cws_ml = ws_ml;
    uint16_t* ob = static_cast<uint16_t*>(out);
    if (D <= 64)
        FORGE_CUDA_TRY(launch_pdl(decode_combine_kernel<64, F16>, dim3(B * Hq), dim3(64), 0, s, cws_o, cws_ml, ob, num_splits, D));
    else
        FORGE_CUDA_TRY(launch_pdl(decode_combine_kernel<128, F16>, dim3(B * Hq), dim3(128), 0, s, cws_o, cws_ml, ob, num_splits, D));
    return finish_launch(1);
}

}  // namespace
}  // namespace forge

extern "C" int forge_attn_decode_splitkv(const void* q, const void* k_cache, const void* v_cache, void* out,
                                         int B, int Hq, int Hkv, int Smax, int D,
                                         const int32_t* lens, int num_splits, float scale,
                                         void* workspace, size_t workspace_bytes, void* stream) {
    return forge::decode_splitkv_impl<false>(q, k_cache, v_cache, out, B, Hq, Hkv, Smax, D, lens, num_splits, scale,
                                             workspace, workspace_bytes, stream);
}

extern "C" int forge_attn_decode_splitkv_f16(const void* q, const void* k_cache, const void* v_cache, void* out,
                                             int B, int Hq, int Hkv, int Smax, int D,
                                             const int32_t* lens, int num_splits, float scale,
                                             void* workspace, size_t workspace_bytes, void* stream) {
    return forge::decode_splitkv_impl<true>(q, k_cache, v_cache, out, B, Hq, Hkv, Smax, D, lens, num_splits, scale,
                                            workspace, workspace_bytes, stream);
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
