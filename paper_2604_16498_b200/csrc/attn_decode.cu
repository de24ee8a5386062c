// Split-KV decode attention with the combine step folded in: Eq. 9 for a single query row per head
// over the first lens[b] rows of a KV cache.  The cached sequence of a (batch, kv head) is cut into
// pieces; each piece yields a partial (running max m, running sum l, unnormalised output) and the
// pieces are merged:
//     M = max_s m_s,   L = sum_s 2^(m_s - M) l_s,   out = sum_s 2^(m_s - M) O_s / L
// (scores are kept in log2 units: they are multiplied by scale * log2(e)).
//
// The work is bound by streaming K and V from HBM once, and HBM only delivers its bandwidth
// with a deep queue of requests (pure streaming with 48 KB in flight per SM reaches 4.2 TB/s on
// this part, with 250 KB 5.8 TB/s).  So the kernel is persistent and every warp is an independent
// worker: it owns whole pieces, keeps a private ring of 16-row blocks in shared memory filled by
// TMA tile copies (16 rows x 64 columns each, 128-byte swizzle, completion counted on an mbarrier
// per stage) that run ahead across piece boundaries (7 warps x 16 KB in flight per SM), and writes
// its partial straight from registers.  No warp ever waits for another one.
//
// Pieces.  All pieces of a call are C blocks of 16 rows long (the last piece of a sequence may be
// shorter).  Every warp works C out for itself from lens: the smallest C that is at least the even
// share of all blocks per worker and at least ceil(longest sequence / num_splits) blocks (so no
// sequence has more than num_splits pieces), raised further, if a modest raise achieves it, until
// there are no more pieces than workers.  Then each worker streams at most one piece of the common
// length, instead of num_splits pieces per sequence whose lengths differ as the sequences do.  With
// more pieces than workers, worker w takes pieces w, w + workers, ...
//
// Combine.  A (batch, kv head) with one piece is normalised and written by its worker.  Otherwise
// each worker writes its partial to the workspace and, with release-acquire ordering, adds one to
// the arrival counter of its (batch, kv head); the worker that brings the counter to the number of
// pieces merges all partials of the G heads, writes the output rows and puts the counter back to
// zero.  Nobody waits: whoever arrives last does the merge.  The counters live at the start of the
// workspace and must be zero when a call starts; every call leaves them at zero.
// The G = Hq / Hkv query heads that share a KV head are processed together, so every cached row
// is read exactly once.  The dot products run on warp-level tensor-core MMAs (m16n8k16) with
// fragments read from the swizzled ring; fp32 FMAs with shuffle reductions were bound by
// instruction issue.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <mutex>

#include "forge_common.cuh"
#include "sm100_ptx.cuh"
#include "tmap.cuh"

namespace forge {
namespace {

// Workers per CTA.  Each keeps its ring full, so the warp count sets how many bytes the SM has in flight; beyond
// what saturates the memory system, more only queue: every block arrives later, the first ones spread over a
// longer start-up burst, and the call ends one loaded latency after its last request.  Measured at B 16,
// 32/8 heads, lengths 1024..4096, D = 128 (148 MB): 5 / 6 / 7 / 8 warps give 33.1 / 31.5 / 31.0 / 33.4 us
// (30.1 / 28.9 / 31.4 us for 6 / 7 / 8 warps once the rows are loaded with the evict-first policy).
constexpr int kWarps = 7;
constexpr int kThreads = kWarps * 32;
constexpr int kBlockKeys = 16;             // cached rows per ring stage
// Per warp.  16 KB (two stages of 16 rows at D = 128) measured a little faster than 24 KB: the memory system is
// saturated either way, and what is queued beyond that only adds to the latency of every block, which is what
// the end of the call (the last blocks of the slowest warps) waits for.
constexpr int kWarpRingBytes = 16 * 1024;
constexpr int kSingleLevelPieces = 32;     // up to this many pieces of a sequence are merged by one warp in one go
                                           // (one (m, l) pair per lane and head)
constexpr int kMergeGroup = 16;            // beyond that: groups of sixteen, then the (at most sixteen) groups' results
constexpr int kMaxSplits = kMergeGroup * kMergeGroup;
constexpr int kPiecesPerLane = 1;          // no merge walks through more than 32 partials

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

// One piece of a (batch, kv head): rows [s0, s1) of its cache, piece number `piece` of `pieces`.
struct Item {
    int b, kvh, piece, pieces, s0, s1;
};

__device__ __forceinline__ int warp_max(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ unsigned warp_sum(unsigned v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// The piece schedule of a call, worked out by every warp for itself (all lanes take part and get the
// same answer): blocks of 16 rows per piece and the number of pieces.  All counts fit 32 bits (the host
// refuses shapes whose block count does not).  Lane l also keeps what the search for a piece needs of
// sequence l (its length, its pieces and the running total up to and including it): with B <= 32 no
// piece lookup touches memory again, which shortens the way from the first read of lens to the first copy.
struct Schedule {
    int C;               // blocks per piece
    unsigned num_items;  // pieces of all (batch, kv head) pairs
    int len0, P0, incl0; // of sequence `lane`: clamped length, pieces, pieces of sequences 0..lane
};
__device__ __forceinline__ int clamped_len(const int32_t* lens, int b, int Smax) { return min(max(lens[b], 0), Smax); }
__device__ __forceinline__ int blocks_of_len(int len) { return (len + kBlockKeys - 1) / kBlockKeys; }
// pieces of a sequence of nb blocks: at least one, so that a sequence without rows still gets its zeros
__device__ __forceinline__ int pieces_of(int nb, int C) { return max((nb + C - 1) / C, 1); }
__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

__device__ __forceinline__ Schedule make_schedule(const int32_t* lens, int B, int Hkv, int Smax, int num_splits,
                                                  int workers, int lane) {
    Schedule s;
    s.len0 = (lane < B) ? clamped_len(lens, lane, Smax) : 0;
    const int nb0 = blocks_of_len(s.len0);
    unsigned total = nb0;
    int max_nb = nb0;
    for (int b = 32 + lane; b < B; b += 32) {
        const int nb = blocks_of_len(clamped_len(lens, b, Smax));
        total += nb;
        max_nb = max(max_nb, nb);
    }
    total = warp_sum(total) * Hkv;
    max_nb = warp_max(max_nb);
    // pieces of all sequences for a piece length C; leaves group 0's scan in s
    auto count = [&](int C) {
        s.P0 = (lane < B) ? pieces_of(nb0, C) : 0;
        s.incl0 = warp_incl_scan(s.P0, lane);
        unsigned n = (unsigned)__shfl_sync(0xffffffffu, s.incl0, 31);
        if (B > 32) {
            unsigned rest = 0;
            for (int b = 32 + lane; b < B; b += 32) rest += pieces_of(blocks_of_len(clamped_len(lens, b, Smax)), C);
            n += warp_sum(rest);
        }
        return n * Hkv;
    };
    const int c_lo = max(max((int)((total + workers - 1) / (unsigned)workers), (max_nb + num_splits - 1) / num_splits), 1);
    s.C = c_lo;
    s.num_items = count(c_lo);
    // more pieces than workers: some worker would stream two.  Look for a slightly longer piece that leaves
    // everyone with at most one (sixteen steps of a sixteenth cover up to twice the length).
    if (s.num_items > (unsigned)workers) {
        int C = c_lo;
        bool found = false;
        for (int i = 0; i < 16 && C < max_nb && !found; ++i) {
            C += max(C >> 4, 1);
            const unsigned n = count(C);
            if (n <= (unsigned)workers) { s.C = C; s.num_items = n; found = true; }
        }
        if (!found) s.num_items = count(c_lo);  // restores group 0's scan for c_lo
    }
    return s;
}

// Piece number idx in dealing order: the kv heads of a piece of rows are consecutive (neighbouring workers
// stream the same rows of different heads), then the next piece of the sequence, then the next sequence.
// A warp-wide scan over lens in groups of 32 sequences finds the sequence (the first group's scan is kept
// in the schedule); all lanes get the same Item.
__device__ __forceinline__ Item make_item(unsigned idx, const Schedule& sc, const int32_t* lens, int B, int Hkv, int Smax,
                                          int lane) {
    Item it;
    const unsigned pc = idx / (unsigned)Hkv;  // piece counter over the sequences
    it.kvh = (int)(idx - pc * (unsigned)Hkv);
    it.b = 0; it.piece = 0; it.pieces = 1; it.s0 = it.s1 = 0;
    const int C = sc.C;
    unsigned cum = 0;
    int len = sc.len0, P = sc.P0, incl = sc.incl0;
    for (int b0 = 0; b0 < B; b0 += 32) {
        if (b0 > 0) {
            len = (b0 + lane < B) ? clamped_len(lens, b0 + lane, Smax) : 0;
            P = (b0 + lane < B) ? pieces_of(blocks_of_len(len), C) : 0;
            incl = warp_incl_scan(P, lane);
        }
        const unsigned tot = (unsigned)__shfl_sync(0xffffffffu, incl, 31);
        if (pc < cum + tot) {
            const unsigned hit = __ballot_sync(0xffffffffu, pc < cum + (unsigned)incl);  // first lane whose range ends beyond pc
            const int src = __ffs(hit) - 1;
            const int len_s = __shfl_sync(0xffffffffu, len, src);
            const int P_s = __shfl_sync(0xffffffffu, P, src);
            const int incl_s = __shfl_sync(0xffffffffu, incl, src);
            it.b = b0 + src;
            it.pieces = P_s;
            it.piece = (int)(pc - (cum + (unsigned)(incl_s - P_s)));
            it.s0 = min(it.piece * C * kBlockKeys, len_s);
            it.s1 = min(it.s0 + C * kBlockKeys, len_s);
            break;
        }
        cum += tot;
    }
    return it;
}

// Merge of `pieces` partials of the G heads of one (batch, kv head), done by the warp that completed the last
// of them: the partials in slots first, first + stride, ...  With `final` the result is normalised and written
// to the output rows; otherwise it is written back, unnormalised, as the partial in slot `first` (the first
// level of a two-level merge).  Lane = D / 32 consecutive output dims.  A function of its own (not inlined):
// it runs once per (batch, kv head) or group of pieces and must not take registers away from the streaming loop.
template <int D, int G, bool F16>
__device__ __forceinline__ void merge_impl(float* __restrict__ ws_o, float* __restrict__ ws_ml,
                                           uint16_t* __restrict__ out, int head0, int first, int stride, int pieces,
                                           bool final, int num_splits, int head_dim, int lane) {
    // The merge sits at the very end of the call (all pieces of a sequence end together), so it is
    // arranged for few round trips to L2: the (m, l) pairs of all heads are requested first, then the
    // partial outputs of two heads and sixteen pieces at a time, all before anything is used.
    constexpr int V = D / 32;  // floats per lane
    const int P = pieces;
    float2 ml[G][kPiecesPerLane];  // (m, l) of pieces lane, lane + 32, ... of every head
#pragma unroll
    for (int h = 0; h < G; ++h) {
        const float2* mlp = reinterpret_cast<const float2*>(ws_ml) + (size_t)(head0 + h) * num_splits + first;
#pragma unroll
        for (int j = 0; j < kPiecesPerLane; ++j)
            ml[h][j] = (lane + 32 * j < P) ? __ldcg(mlp + (lane + 32 * j) * stride) : make_float2(-INFINITY, 0.f);
    }
    auto load_part = [&](int h, int sp, float (&dst)[V]) {
        const float* src = ws_o + ((size_t)(head0 + h) * num_splits + first + sp * stride) * D + lane * V;
        if constexpr (V == 4) {
            const float4 t4 = __ldcg(reinterpret_cast<const float4*>(src));
            dst[0] = t4.x; dst[1] = t4.y; dst[2] = t4.z; dst[3] = t4.w;
        } else {
            const float2 t2 = __ldcg(reinterpret_cast<const float2*>(src));
            dst[0] = t2.x; dst[1] = t2.y;
        }
    };
#pragma unroll
    for (int h0 = 0; h0 < G; h0 += 2) {
        constexpr int kChunk = 16;
        float part[2][kChunk][V];
        auto load_chunk = [&](int s0) {
#pragma unroll
            for (int e = 0; e < 2; ++e)
#pragma unroll
                for (int i = 0; i < kChunk; ++i) {
                    if (h0 + e < G && s0 + i < P) load_part(h0 + e, s0 + i, part[e][i]);
                    else {
#pragma unroll
                        for (int v = 0; v < V; ++v) part[e][i][v] = 0.f;
                    }
                }
        };
        load_chunk(0);
        // weights of the two heads' pieces: w = 2^(m - M), 0 for a piece without rows
        float w[2][kPiecesPerLane], L[2], Mx[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int h = (h0 + e < G) ? h0 + e : h0;
            float M = ml[h][0].x;
#pragma unroll
            for (int j = 1; j < kPiecesPerLane; ++j) M = fmaxf(M, ml[h][j].x);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
            const float Mr = (M == -INFINITY) ? 0.f : M;
            float l = 0.f;
#pragma unroll
            for (int j = 0; j < kPiecesPerLane; ++j) {
                w[e][j] = exp2f(ml[h][j].x - Mr);
                l = fmaf(w[e][j], ml[h][j].y, l);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
            L[e] = l;
            Mx[e] = M;
        }
        float o_acc[2][V];
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
            for (int v = 0; v < V; ++v) o_acc[e][v] = 0.f;
        for (int s0 = 0; s0 < P; s0 += kChunk) {
            if (s0 > 0) load_chunk(s0);
            // the weights of pieces s0 .. s0 + 15 sit in entry s0 / 32 of their lanes (no dynamic indexing)
            float wsel[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                wsel[e] = w[e][0];
#pragma unroll
                for (int j = 1; j < kPiecesPerLane; ++j) wsel[e] = ((s0 >> 5) == j) ? w[e][j] : wsel[e];
            }
#pragma unroll
            for (int e = 0; e < 2; ++e)
#pragma unroll
                for (int i = 0; i < kChunk; ++i) {
                    const int sp = s0 + i;
                    const float wgt = __shfl_sync(0xffffffffu, wsel[e], sp & 31);
                    if (sp < P && wgt != 0.f) {
#pragma unroll
                        for (int v = 0; v < V; ++v) o_acc[e][v] = fmaf(wgt, part[e][i][v], o_acc[e][v]);
                    }
                }
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            if (h0 + e >= G) continue;
            if (!final) {  // the merged partial (M, L, sum of the weighted partial outputs) takes the first slot
                const size_t slot = (size_t)(head0 + h0 + e) * num_splits + first;
                float* dst = ws_o + slot * D + lane * V;
                if constexpr (V == 4) *reinterpret_cast<float4*>(dst) = make_float4(o_acc[e][0], o_acc[e][1], o_acc[e][2], o_acc[e][3]);
                else *reinterpret_cast<float2*>(dst) = make_float2(o_acc[e][0], o_acc[e][1]);
                if (lane == 0) *reinterpret_cast<float2*>(ws_ml + slot * 2) = make_float2(Mx[e], L[e]);
                continue;
            }
            const float invL = L[e] > 0.f ? 1.f / L[e] : 0.f;
            uint16_t* orow = out + (size_t)(head0 + h0 + e) * head_dim + lane * V;
            if (lane * V < head_dim) {  // head_dim is a multiple of 8, V divides 8: all V dims are inside or none
                if constexpr (V == 4)
                    *reinterpret_cast<uint2*>(orow) = make_uint2(pack16x2<F16>(o_acc[e][0] * invL, o_acc[e][1] * invL),
                                                                 pack16x2<F16>(o_acc[e][2] * invL, o_acc[e][3] * invL));
                else
                    *reinterpret_cast<uint32_t*>(orow) = pack16x2<F16>(o_acc[e][0] * invL, o_acc[e][1] * invL);
            }
        }
    }
}

// The common case: all pieces of a (batch, kv head), at most 32, merged into the output rows.
template <int D, int G, bool F16>
__device__ __noinline__ void merge_pieces(float* __restrict__ ws_o, float* __restrict__ ws_ml,
                                          uint16_t* __restrict__ out, int head0, int pieces, int num_splits,
                                          int head_dim, int lane) {
    merge_impl<D, G, F16>(ws_o, ws_ml, out, head0, 0, 1, pieces, true, num_splits, head_dim, lane);
}

// Arrival and merge for a sequence cut into more than 32 pieces (a long sequence in a small batch): two levels,
// so that the merge work is spread over as many warps as there are groups of sixteen pieces and no warp walks
// through more than sixteen partials per level.  The last arrival of a group of sixteen merges them into the
// group's first slot and then arrives at the (batch, kv head)'s counter; the last of those merges the groups'
// results.  The arrivals are the same release-acquire read-modify-writes as in the kernel.
template <int D, int G, bool F16>
__device__ __noinline__ void arrive_two_level(unsigned int* __restrict__ counters, float* __restrict__ ws_o,
                                              float* __restrict__ ws_ml, uint16_t* __restrict__ out, int B, int Hkv,
                                              int b, int kvh, int piece, int pieces, int head0, int num_splits,
                                              int head_dim, int lane) {
    auto arrive = [&](unsigned int* counter) {
        __syncwarp();
        unsigned int arrived = 0;
        if (lane == 0)
            asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(arrived) : "l"(counter) : "memory");
        return __shfl_sync(0xffffffffu, arrived, 0);
    };
    unsigned int* group_counter = counters + b * Hkv + kvh;
    const int sg = piece / kMergeGroup, n_sg = (pieces + kMergeGroup - 1) / kMergeGroup;
    const int in_sg = min(kMergeGroup, pieces - sg * kMergeGroup);
    unsigned int* sg_counter = counters + B * Hkv + (b * Hkv + kvh) * (kMaxSplits / kMergeGroup) + sg;
    if (arrive(sg_counter) + 1 != (unsigned)in_sg) return;
    if (lane == 0) *sg_counter = 0;  // as the next call expects it
    merge_impl<D, G, F16>(ws_o, ws_ml, out, head0, sg * kMergeGroup, 1, in_sg, false, num_splits, head_dim, lane);
    if (arrive(group_counter) + 1 != (unsigned)n_sg) return;
    if (lane == 0) *group_counter = 0;
    merge_impl<D, G, F16>(ws_o, ws_ml, out, head0, 0, kMergeGroup, n_sg, true, num_splits, head_dim, lane);
}

// Worker w (= warp) takes pieces w, w + workers, ...; consecutive pieces go to different SMs.
//   S[head, key]  = Q K^T   as m16n8k16 with A = Q (rows = the G heads, padded with zero rows) and
//                   B = K rows (the contraction runs over the head dimension in whatever order the
//                   16-byte chunks deliver it, the same for Q and K);
//   online softmax on the accumulator fragment (lane (g, c) owns head g, keys 2c, 2c+1 of each 8);
//   O^T[dim, head] += V^T P^T  with A = pairs of V rows interleaved with byte permutes and B = the
//                   probabilities exactly where the first MMA left them.
// Workspace: counters[B * Hkv] and counters of the groups of sixteen pieces [B * Hkv][16] (zero between calls), then ws_o[(b, head, piece)][D] and ws_ml[(b, head, piece)][2]
// with num_splits piece slots per (batch, head).
template <int D, int G, bool F16>
__global__ void __launch_bounds__(kThreads, 1)
decode_split_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                    const uint16_t* __restrict__ q, const int32_t* __restrict__ lens, uint16_t* __restrict__ out,
                    unsigned int* __restrict__ counters, float* __restrict__ ws_o, float* __restrict__ ws_ml,
                    int B, int Hq, int Hkv, int Smax, int head_dim, int num_splits, float scale_log2, int* status) {
    constexpr int NKB = D / 32;  // 32-dim blocks of the head dimension (two k16 MMAs each)
    constexpr int NHB = D / 64;  // 64-dim blocks of the output (four 16-dim MMAs each)
    // A stage holds 16 rows of K and 16 rows of V as D / 64 tiles of 16 rows x 128 bytes each; 16-byte chunk
    // k of row r of a tile sits at r * 128 + ((k ^ (r & 7)) << 4) (the TMA unit's 128-byte swizzle).
    constexpr int kTileBytes = kBlockKeys * 128;
    constexpr int kKBytes = (D / 64) * kTileBytes;
    constexpr int kStageBytes = 2 * kKBytes;
    constexpr int kStages = kWarpRingBytes / kStageBytes;  // 2 for D = 128, 4 for D = 64
    static_assert(kStages >= 2 && kStages <= 8, "ring size");

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
    // Set-up done: the next kernel in the stream may move in as SMs free up.  Nothing global is touched
    // before the previous kernel has completed and its writes are visible.
    pdl_launch_dependents();
    pdl_wait();

    const int workers = gridDim.x * kWarps;
    const int worker = warp * gridDim.x + blockIdx.x;
    const Schedule sched = make_schedule(lens, B, Hkv, Smax, num_splits, workers, lane);
    const unsigned num_items = sched.num_items;
    auto item_of_round = [&](int r) { return (unsigned)r * (unsigned)workers + (unsigned)worker; };

    // ---- prefetch cursor: runs kStages blocks ahead of the compute, across item boundaries (a stage is
    // refilled as soon as its fragments are in registers, before the MMAs on them)
    int p_round = 0, p_j0 = 0, p_s1 = 0;
    unsigned p_idx = item_of_round(0);
    int p_bk = 0;  // batch * Hkv + kv head of the cursor's item
    int p_n = 0;  // blocks issued
    auto p_open = [&]() {  // position the cursor on the first block of the next non-empty item
        while (p_idx < num_items) {
            const Item it = make_item(p_idx, sched, lens, B, Hkv, Smax, lane);
            if (it.s1 > it.s0) {
                p_j0 = it.s0;
                p_s1 = it.s1;
                p_bk = it.b * Hkv + it.kvh;
                return;
            }
            p_idx = item_of_round(++p_round);
        }
    };
    // Every cached row is read once per call: its lines are marked first to go, so that they do not push the
    // partials, the queries and whatever the caller keeps in L2 out of it (2 us of 31 at B 16, lengths 1024..4096).
    const uint64_t stream_policy = ptx::l2_policy_evict_first();
    auto issue = [&]() {  // one lane starts the block's tile copies (rows past the cache's end are zero-filled)
        if (p_idx < num_items) {
            if (lane == 0) {
                const int st = p_n % kStages;
                const uint32_t dst = ring + st * kStageBytes;
                ptx::mbar_expect_tx(&full[st], kStageBytes);
#pragma unroll
                for (int cb = 0; cb < D / 64; ++cb) {
                    ptx::tma_load_3d_addr_hint(dst + cb * kTileBytes, &tmap_k, &full[st], cb * 64, p_j0, p_bk, stream_policy);
                    ptx::tma_load_3d_addr_hint(dst + kKBytes + cb * kTileBytes, &tmap_v, &full[st], cb * 64, p_j0, p_bk, stream_policy);
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

    Item nxt = {0, 0, 0, 1, 0, 0};
    uint32_t qn[NKB][4];
    if (item_of_round(0) < num_items) {
        nxt = make_item(item_of_round(0), sched, lens, B, Hkv, Smax, lane);
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
            nxt = make_item(item_of_round(round + 1), sched, lens, B, Hkv, Smax, lane);
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
        // ---- the piece is done.  This lane holds, of heads 2c and 2c+1, dims hb*64 + g*8 + {0..7}.
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        const int head0 = it.b * Hq + it.kvh * G;  // first query head of the group, as a row of q / out
        if (it.pieces == 1) {
            // the only piece of its (batch, kv head): normalise and write the output rows (zeros without rows)
            const float l_even = __shfl_sync(0xffffffffu, l_run, (2 * c) * 4);
            const float l_odd = __shfl_sync(0xffffffffu, l_run, (2 * c + 1) * 4);
            const float inv[2] = {l_even > 0.f ? 1.f / l_even : 0.f, l_odd > 0.f ? 1.f / l_odd : 0.f};
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (2 * c + e >= G) continue;
                uint16_t* orow = out + (size_t)(head0 + 2 * c + e) * head_dim;
#pragma unroll
                for (int hb = 0; hb < NHB; ++hb) {
                    const int d0 = hb * 64 + g * 8;
                    if (d0 >= head_dim) continue;  // padding columns of a head size below the kernel's
                    uint32_t w[4];
#pragma unroll
                    for (int t = 0; t < 4; t += 2) {  // dims d0 + t, t+1 (acc[.][t][e], acc[.][t+1][e]) and d0 + 4 + t, t+1
                        w[t / 2] = pack16x2<F16>(acc[hb][t][e] * inv[e], acc[hb][t + 1][e] * inv[e]);
                        w[2 + t / 2] = pack16x2<F16>(acc[hb][t][2 + e] * inv[e], acc[hb][t + 1][2 + e] * inv[e]);
                    }
                    *reinterpret_cast<uint4*>(orow + d0) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            continue;
        }
        // ---- several pieces: partial to the workspace, then the arrival count
        const size_t slot0 = (size_t)head0 * num_splits + it.piece;  // head 0 of the group
        if (g < G && c == 0) {
            ws_ml[(slot0 + (size_t)g * num_splits) * 2] = m_run;
            ws_ml[(slot0 + (size_t)g * num_splits) * 2 + 1] = l_run;
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            if (2 * c + e >= G) continue;
            float* o = ws_o + (slot0 + (size_t)(2 * c + e) * num_splits) * D;
#pragma unroll
            for (int hb = 0; hb < NHB; ++hb) {
                const int d0 = hb * 64 + g * 8;
                *reinterpret_cast<float4*>(o + d0) = make_float4(acc[hb][0][e], acc[hb][1][e], acc[hb][2][e], acc[hb][3][e]);
                *reinterpret_cast<float4*>(o + d0 + 4) =
                    make_float4(acc[hb][0][2 + e], acc[hb][1][2 + e], acc[hb][2][2 + e], acc[hb][3][2 + e]);
            }
        }
        if (it.pieces > kSingleLevelPieces) {
            arrive_two_level<D, G, F16>(counters, ws_o, ws_ml, out, B, Hkv, it.b, it.kvh, it.piece, it.pieces, head0,
                                        num_splits, head_dim, lane);
            continue;
        }
        // The arrival is a release-acquire read-modify-write at device scope by lane 0, after a warp barrier:
        // the warp's stores of the partial happen before it, and whoever reads the full count has acquired the
        // partials of all earlier arrivals.  (One combined operation instead of fence, atomic, fence: the
        // round trips to L2 at this point are what the end of the call waits for.)
        __syncwarp();
        unsigned int arrived = 0;
        if (lane == 0)
            asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(arrived) : "l"(counters + it.b * Hkv + it.kvh) : "memory");
        arrived = __shfl_sync(0xffffffffu, arrived, 0);  // the other lanes read the partials after this exchange
        if (arrived + 1 != (unsigned)it.pieces) continue;

        // ---- last to arrive: merge the pieces of the G heads
        if (lane == 0) counters[it.b * Hkv + it.kvh] = 0;  // as the next call expects it
        merge_pieces<D, G, F16>(ws_o, ws_ml, out, head0, it.pieces, num_splits, head_dim, lane);
    }
    if (failed) {
        if (lane == 0) atomicExch(status, 1);
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies in flight land before the ring goes away
    }
}

template <int D, int G, bool F16>
int launch_split(const void* q, const void* kc, const void* vc, const int32_t* lens, void* out, unsigned int* counters,
                 float* ws_o, float* ws_ml, int B, int Hq, int Hkv, int Smax, int head_dim, int num_splits,
                 float scale_log2, cudaStream_t s) {
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
    // no more pieces than this can exist, whatever lens holds
    const long long blocks_max = (Smax + kBlockKeys - 1) / kBlockKeys;
    const long long items = (long long)B * Hkv * (blocks_max < num_splits ? blocks_max : num_splits);
    const long long ctas = (items + kWarps - 1) / kWarps;
    const int grid = ctas < sms ? (int)ctas : sms;
    FORGE_CUDA_TRY(launch_pdl(kernel, dim3(grid), dim3(kThreads), kSmem, s, tk, tv, static_cast<const uint16_t*>(q),
                              lens, static_cast<uint16_t*>(out), counters, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim,
                              num_splits, scale_log2, status));
    return finish_launch(1);
}

template <int D, bool F16>
int dispatch_g(int G, const void* q, const void* kc, const void* vc, const int32_t* lens, void* out,
               unsigned int* counters, float* ws_o, float* ws_ml, int B, int Hq, int Hkv, int Smax, int head_dim,
               int num_splits, float scale_log2, cudaStream_t s) {
#define FORGE_DECODE_CASE(g)                                                                                     \
    case g:                                                                                                      \
        return launch_split<D, g, F16>(q, kc, vc, lens, out, counters, ws_o, ws_ml, B, Hq, Hkv, Smax, head_dim, \
                                       num_splits, scale_log2, s)
    switch (G) {
        FORGE_DECODE_CASE(1);
        FORGE_DECODE_CASE(2);
        FORGE_DECODE_CASE(3);
        FORGE_DECODE_CASE(4);
        FORGE_DECODE_CASE(5);
        FORGE_DECODE_CASE(6);
        FORGE_DECODE_CASE(7);
        FORGE_DECODE_CASE(8);
        default: return FORGE_ERR_UNSUPPORTED;
    }
#undef FORGE_DECODE_CASE
}

// Bytes of the arrival counters at the start of the workspace: one per (batch, kv head) and, behind those, one
// per group of sixteen pieces of a (batch, kv head) for the two-level merge; sized for Hkv = Hq.
// At least 1088 KiB, so that every shape with B * Hq <= 16384 keeps its counters (and only counters) in the
// same region: a workspace cleared once then serves calls of any such shape.
inline size_t counter_bytes(int B, int Hq) {
    constexpr size_t kPerHead = (1 + kMaxSplits / kMergeGroup) * sizeof(unsigned int);
    const size_t need = ((size_t)B * Hq * kPerHead + 255) & ~(size_t)255;
    return need > 16384 * kPerHead ? need : 16384 * kPerHead;
}

}  // namespace
}  // namespace forge

extern "C" size_t forge_attn_decode_workspace_bytes(int B, int Hq, int D, int num_splits) {
    if (B <= 0 || Hq <= 0 || D <= 0 || num_splits <= 0) return 0;
    const size_t slots = (size_t)B * Hq * num_splits;
    const int dp = D <= 64 ? 64 : 128;  // the partial outputs are as wide as the kernel's head dimension
    return forge::counter_bytes(B, Hq) + ((slots * (size_t)(dp + 2) * sizeof(float) + 15) & ~(size_t)15);
}

extern "C" int forge_attn_decode_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    using namespace forge;
    if (!workspace || workspace_bytes == 0) return FORGE_ERR_INVALID_ARG;
    FORGE_CUDA_TRY(cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)));
    return FORGE_OK;
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
    if (num_splits > kMaxSplits || Hkv > 65535 || B > 65535) return FORGE_ERR_UNSUPPORTED;
    // the kernel counts 16-row blocks and pieces in 32 bits
    if ((long long)B * Hkv * ((Smax + kBlockKeys - 1) / kBlockKeys) >= (1LL << 31)) return FORGE_ERR_UNSUPPORTED;
    if (!workspace || !aligned16(workspace)) return FORGE_ERR_INVALID_ARG;
    if (workspace_bytes < forge_attn_decode_workspace_bytes(B, Hq, D, num_splits)) return FORGE_ERR_WORKSPACE;

    const size_t slots = (size_t)B * Hq * num_splits;
    unsigned int* counters = static_cast<unsigned int*>(workspace);
    float* ws_o = reinterpret_cast<float*>(static_cast<char*>(workspace) + counter_bytes(B, Hq));
    float* ws_ml = ws_o + slots * (D <= 64 ? 64 : 128);
    const float scale_log2 = scale * 1.4426950408889634f;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int G = Hq / Hkv;
    return (D <= 64) ? dispatch_g<64, F16>(G, q, k_cache, v_cache, lens, out, counters, ws_o, ws_ml, B, Hq, Hkv, Smax, D, num_splits, scale_log2, s)
                     : dispatch_g<128, F16>(G, q, k_cache, v_cache, lens, out, counters, ws_o, ws_ml, B, Hq, Hkv, Smax, D, num_splits, scale_log2, s);
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
    // the arrival counters and the partials of this problem (num_splits slots of (D <= 64 ? 64 : 128) + 2 floats per
    // (batch, head)) must fit the fixed array
    const size_t need = forge_attn_decode_workspace_bytes(B, Hq, D, num_splits);
    if (need > (size_t)FORGE_DECODE_STATIC_SCRATCH_BYTES) return FORGE_ERR_WORKSPACE;
    if (!q || !k_cache || !v_cache || !out || !lens) return FORGE_ERR_INVALID_ARG;
    void* scratch = static_scratch_for_current_device();
    if (!scratch) return FORGE_ERR_CUDA;
    return forge_attn_decode_splitkv(q, k_cache, v_cache, out, B, Hq, Hkv, Smax, D, lens, num_splits, scale,
                                     scratch, (size_t)FORGE_DECODE_STATIC_SCRATCH_BYTES, stream);
}
