// Fused Linear + bias + activation (+ residual) on CTA pairs (Listing 6 / Eq. 11, the same operator as
// linear_gelu.cu).  Why a second kernel: the one-CTA kernel is bound by the rate at which an SM can pull
// operands out of L2 (a 128 x 192 tile reads 40 KB per 64-deep k-step for 384 tensor-core cycles, more
// than the SM's L2 port delivers).  Here two CTAs on neighbouring SMs (a cluster of two) share one
// 256 x 256 output tile: each loads its own 128 rows of X and its own 128 columns of W, with its own TMA
// copies (no multicast), and the tensor cores of both SMs read both halves of W (tcgen05.mma
// cta_group::2).  Per SM and k-step that is 32 KB for 512 tensor-core cycles: 64 B per cycle instead of 104.
//
// Roles per CTA (576 threads):
//   warp 0    : TMA producer for this CTA's operand halves; the bytes of both CTAs are counted on the even
//               CTA's barrier of the stage, so the issuer observes one barrier per k-step
//   warp 1    : even CTA: issues the pair's MMAs (one elected lane).  In both CTAs this warp allocates and
//               frees the tensor memory.
//   warps 2-17: epilogue of this CTA's 128 x 256 half of the tile; each warp on its own (no barriers)
// Two accumulators of 256 columns: the epilogue of tile i overlaps the main loop of tile i + 1.
// Gated form (SwiGLU, silu(X Wg) * (X Wu)): the pair's tile is 256 rows x 128 output columns; each CTA loads 64
// gate columns and the 64 up columns of the same outputs, so the accumulator holds [gate | up] of CTA 0's columns,
// then [gate | up] of CTA 1's, and the epilogue multiplies the two halves as it reads them back.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "activations.cuh"
#include "forge_common.cuh"
#include "linear_pair.cuh"
#include "sm100_ptx.cuh"
#include "tmap.cuh"

namespace forge {
namespace {

using namespace ptx;

constexpr int kBM = 128;          // rows per CTA
constexpr int kBN = 256;          // columns of the pair's tile (128 loaded per CTA)
constexpr int kBK = 64;
constexpr int kStages = 5;
constexpr int kEpiWarps = 16;     // four per TMEM lane quarter, one 64-column block of the tile each
constexpr int kThreads = 64 + kEpiWarps * 32;
constexpr int kTmemCols = 512;    // two accumulators of 256 columns

struct PairSmem {
    static constexpr int kABytes = kBM * kBK * 2;          // 16 KB: 128 rows of X
    static constexpr int kBBytes = kBK * (kBN / 2) * 2;    // 16 KB: 128 columns of W
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kOutBytes = kEpiWarps * 4096;     // output staging: 32 rows x 64 elements per epilogue warp
    static constexpr int kOutOffset = kStages * kStageBytes;
    static constexpr int kBarOffset = kOutOffset + kOutBytes;
    // full[S], empty[S], tmem_full[2], tmem_empty[2]; then the TMEM base
    static constexpr int kNumBars = 2 * kStages + 4;
    static constexpr int kTotal = kBarOffset + kNumBars * 8 + 16;
    static constexpr int kAlloc = kTotal + 1024;
};

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
template <bool F16>
__device__ __forceinline__ float widen16(uint16_t bits) {
    if constexpr (F16) return __half2float(__ushort_as_half(bits));
    else return __uint_as_float(static_cast<uint32_t>(bits) << 16);
}

// GATED: tmap_w = gate weights, tmap_w2 = up weights, tmap_y stores boxes of 32 columns; no bias, residual or ACT.
template <int ACT, bool W_NK, bool F16, bool GATED>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
linear_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                   const __grid_constant__ CUtensorMap tmap_w2,
                   const __grid_constant__ CUtensorMap tmap_y, const uint16_t* __restrict__ bias,
                   const uint16_t* __restrict__ residual, int M, int N, int K, int* __restrict__ status) {
    using L = PairSmem;
    extern __shared__ uint8_t smem_raw[];
    // the same offset in both CTAs (the dynamic shared memory of a kernel starts at the same address in each)
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);  // even CTA: both CTAs' operands of a stage have landed
    uint64_t* empty = full + kStages;                                   // the pair's MMAs have read the stage
    uint64_t* tmem_full = empty + kStages;
    uint64_t* tmem_empty = tmem_full + 2;                               // even CTA: both epilogues have read the accumulator
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0: issues the MMAs
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    constexpr int BNO = GATED ? kBN / 2 : kBN;  // output columns of the pair's tile
    const int tiles_m = (M + 2 * kBM - 1) / (2 * kBM), tiles_n = (N + BNO - 1) / BNO;
    const int num_tiles = tiles_m * tiles_n;
    const int kblocks = (K + kBK - 1) / kBK;
    // Work units.  The tiles of the last, incomplete round of the persistent schedule are cut into two halves of
    // 128 columns when that lets them all run at once: the round then takes half as long, which matters when a
    // pair only gets five or six tiles in all.  (Not for the gated form: a CTA's half would be 32 + 32 columns.)
    const int rem = num_tiles % num_pairs;
    const bool split = !GATED && rem > 0 && 2 * rem <= num_pairs;
    const int n_whole = split ? num_tiles - rem : num_tiles;
    const int num_units = n_whole + (split ? 2 * rem : 0);
    struct Unit { int tile, col0, width; };  // col0: first column of the unit inside its tile
    auto unit_of = [&](int u) {
        Unit x;
        if (u < n_whole) { x.tile = u; x.col0 = 0; x.width = BNO; }
        else { const int v = u - n_whole; x.tile = n_whole + (v >> 1); x.col0 = (v & 1) * (kBN / 2); x.width = kBN / 2; }
        return x;
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&tmem_full[i], 1); mbar_init(&tmem_empty[i], 2 * kEpiWarps); }
        fence_mbar_init();
        prefetch_tmap(&tmap_x);
        prefetch_tmap(&tmap_w);
        if constexpr (GATED) prefetch_tmap(&tmap_w2);
        prefetch_tmap(&tmap_y);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_base_slot, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();  // both CTAs' barriers exist before anyone signals across
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;
    bool failed = false;
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            for (int u = pair; u < num_units && !failed; u += num_pairs) {
                const Unit un = unit_of(u);
                const int tile = un.tile;
                const int m0 = (tile / tiles_n) * 2 * kBM + (int)rank * kBM;
                // this CTA's columns of W: half of the unit's (gated: 64 gate columns and the same 64 up columns)
                const int n0 = (tile % tiles_n) * BNO + un.col0 + (int)rank * (un.width / 2);
                const bool narrow = un.width < BNO;  // a half tile: 64 columns of W per CTA
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&empty[stage], phase ^ 1)) { failed = true; break; }
                    uint8_t* sa = smem + stage * L::kStageBytes;
                    uint8_t* sb = sa + L::kABytes;
                    // one arrival and the bytes of BOTH CTAs' tiles, announced by the even CTA on its barrier
                    if (rank == 0) mbar_expect_tx(&full[stage], 2 * (L::kABytes + (narrow ? L::kBBytes / 2 : L::kBBytes)));
                    const uint32_t bar = map_to_cta(&full[stage], 0);
                    tma_load_2d_pair(sa, &tmap_x, bar, kb * kBK, m0);
                    if constexpr (W_NK) {  // rows of W, 64 K-elements (one swizzle span) each
                        if constexpr (GATED) {
                            tma_load_2d_pair(sb, &tmap_w, bar, kb * kBK, n0);               // 64 gate rows
                            tma_load_2d_pair(sb + 64 * 128, &tmap_w2, bar, kb * kBK, n0);   // 64 up rows
                        } else {                                                             // one or two boxes of 64 rows
                            tma_load_2d_pair(sb, &tmap_w, bar, kb * kBK, n0);
                            if (!narrow) tma_load_2d_pair(sb + 64 * 128, &tmap_w, bar, kb * kBK, n0 + 64);
                        }
                    } else {               // boxes of 64 K-rows x 64 columns
                        tma_load_2d_pair(sb, &tmap_w, bar, n0, kb * kBK);
                        if constexpr (GATED) tma_load_2d_pair(sb + kBK * 128, &tmap_w2, bar, n0, kb * kBK);
                        else if (!narrow) tma_load_2d_pair(sb + kBK * 128, &tmap_w, bar, n0 + 64, kb * kBK);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1 && rank == 0) {
        // ------------------------------------------------------------------ even CTA: MMA issuer of the pair
        if (elect_one()) {
            constexpr uint32_t idesc_whole = F16 ? make_idesc_f16(2 * kBM, kBN, /*a_mn_major=*/false, /*b_mn_major=*/!W_NK)
                                                 : make_idesc_bf16(2 * kBM, kBN, /*a_mn_major=*/false, /*b_mn_major=*/!W_NK);
            constexpr uint32_t idesc_half = F16 ? make_idesc_f16(2 * kBM, kBN / 2, false, !W_NK)
                                                : make_idesc_bf16(2 * kBM, kBN / 2, false, !W_NK);
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            for (int u = pair; u < num_units && !failed; u += num_pairs, ++it) {
                const uint32_t idesc = (!GATED && unit_of(u).width < kBN) ? idesc_half : idesc_whole;
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!mbar_wait_cluster(&tmem_empty[acc], acc_phase ^ 1)) { failed = true; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * kBN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait_cluster(&full[stage], phase)) { failed = true; break; }
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
                    const uint32_t sb = sa + L::kABytes;
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        const uint64_t a_desc = make_smem_desc(sa + k * 32, 16, 1024);
                        const uint64_t b_desc = W_NK ? make_smem_desc(sb + k * 32, 16, 1024)
                                                     : make_smem_desc(sb + k * 2048, kBK * 128, 1024);
                        mma_ss_pair(d_tmem, a_desc, b_desc, idesc, (kb | k) != 0);
                    }
                    mma_commit_pair(&empty[stage], 0x3);  // both CTAs' stages are free once these MMAs have read them
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
                if (failed) break;
                mma_commit_pair(&tmem_full[acc], 0x3);    // both epilogues may read the accumulator
            }
        }
    } else if (warp >= 2) {
        // ------------------------------------------------------------------ epilogue of this CTA's 128 rows
        // Every warp works alone: it owns 32 rows (its TMEM lane quarter) of one of the tile's four 64-column
        // blocks, its own 4 KB of staging and its own TMA stores, so the sixteen warps never meet at a barrier.
        const int quarter = warp & 3;    // TMEM lane quarter this warp may access
        const int blk = (warp - 2) >> 2; // its 64-column block of the tile
        uint8_t* stage_out = smem + L::kOutOffset + (warp - 2) * 4096;
        const uint32_t empty_on_leader = map_to_cta(&tmem_empty[0], 0);  // [acc] at + 8 * acc
        int it = 0;
        for (int u = pair; u < num_units; u += num_pairs, ++it) {
            const Unit un = unit_of(u);
            const int tile = un.tile;
            const int m0 = (tile / tiles_n) * 2 * kBM + (int)rank * kBM, n0 = (tile % tiles_n) * BNO + un.col0;
            const int acc = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1;
            if (!warp_wait(&tmem_full[acc], acc_phase)) { failed = true; break; }
            tc_fence_after_sync();
            const int row = quarter * 32 + lane;  // row of this CTA's half of the tile = TMEM lane
            const uint32_t taddr = tmem_base + acc * kBN + (static_cast<uint32_t>(quarter * 32) << 16);
            if (!GATED && blk * 64 >= un.width) {  // a half tile has no block for this warp: only the accumulator hand-back
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(empty_on_leader + acc * 8);
                continue;
            }
            if (lane == 0) tma_store_wait_read<0>();  // this warp's previous store has read the staging rows
            __syncwarp();
            if constexpr (GATED) {
                // This warp: 32 of the tile's 128 output columns.  Output column c of the tile was computed by CTA
                // c / 64, whose part of the accumulator is [gate 64 | up 64] at column (c / 64) * 128.
                const int oc = blk * 32;                                   // first output column of this warp
                const uint32_t gcol = (oc >> 6) * 128 + (oc & 63);         // its gate columns in the accumulator
                uint32_t rg[32], ru[32];
                tmem_ld_x32(taddr + gcol, rg);
                tmem_ld_x32(taddr + gcol + 64, ru);
                tmem_ld_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(empty_on_leader + acc * 8);
#pragma unroll
                for (int c = 0; c < 4; ++c) {  // 16-byte chunk c of this warp's 64-byte staging row
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int k = c * 8 + 2 * i;
                        w[i] = pack16<F16>(activate<FORGE_ACT_SILU>(__uint_as_float(rg[k])) * __uint_as_float(ru[k]),
                                           activate<FORGE_ACT_SILU>(__uint_as_float(rg[k + 1])) * __uint_as_float(ru[k + 1]));
                    }
                    *reinterpret_cast<uint4*>(stage_out + lane * 64 + c * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && m0 + quarter * 32 < M && n0 + oc < N) {
                    tma_store_2d(&tmap_y, stage_out, n0 + oc, m0 + quarter * 32);  // a plain box of 32 columns x 32 rows
                    tma_store_commit();
                }
                continue;
            }
#pragma unroll
            for (int half = 0; half < 2; ++half) {  // 32 columns at a time keeps the registers of 576 threads in bounds
                uint32_t r[32];
                tmem_ld_x32(taddr + blk * 64 + half * 32, r);
                tmem_ld_wait();
                if (half == 1) {
                    // this warp has read all it needs of the accumulator: tell the issuer (in the even CTA)
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(empty_on_leader + acc * 8);
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {  // 16-byte chunk half*4 + c of the row's 128-byte line: 8 columns
                    const int gcol = n0 + blk * 64 + half * 32 + c * 8;
                    uint4 bv = make_uint4(0, 0, 0, 0), res = make_uint4(0, 0, 0, 0);
                    if (bias != nullptr && gcol < N) bv = __ldg(reinterpret_cast<const uint4*>(bias + gcol));
                    if (residual != nullptr && m0 + row < M && gcol < N)
                        res = *reinterpret_cast<const uint4*>(residual + (size_t)(m0 + row) * N + gcol);
                    const uint32_t bw[4] = {bv.x, bv.y, bv.z, bv.w}, rw[4] = {res.x, res.y, res.z, res.w};
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float z0 = __uint_as_float(r[c * 8 + 2 * i]) + widen16<F16>(static_cast<uint16_t>(bw[i] & 0xffffu));
                        const float z1 = __uint_as_float(r[c * 8 + 2 * i + 1]) + widen16<F16>(static_cast<uint16_t>(bw[i] >> 16));
                        w[i] = pack16<F16>(activate<ACT>(z0) + widen16<F16>(static_cast<uint16_t>(rw[i] & 0xffffu)),
                                           activate<ACT>(z1) + widen16<F16>(static_cast<uint16_t>(rw[i] >> 16)));
                    }
                    *reinterpret_cast<uint4*>(stage_out + lane * 128 + (((half * 4 + c) ^ (lane & 7)) << 4)) =
                        make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && m0 + quarter * 32 < M) {
                tma_store_2d(&tmap_y, stage_out, n0 + blk * 64, m0 + quarter * 32);  // rows >= M, columns >= N are clipped
                tma_store_commit();
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    }

    if (failed) {
        atomicExch(status, 1);
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies and MMAs in flight land
    }
    // Neither CTA may leave while the other can still read its shared memory (the MMAs read both halves of W)
    // or signal its barriers.
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

template <int ACT, bool W_NK, bool F16, bool GATED = false>
int launch_pair(const void* x, const void* w, const void* b, const void* residual, void* y, int M, int N, int K,
                cudaStream_t s, const void* w_up = nullptr) {
    using L = PairSmem;
    constexpr int BNO = GATED ? kBN / 2 : kBN;
    CUtensorMap tmap_x, tmap_w, tmap_w2, tmap_y;
    {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
        const uint64_t strides[1] = {(uint64_t)K * 2};
        const uint32_t box[2] = {kBK, kBM};
        if (!encode_tmap_bf16_sw128(&tmap_x, x, 2, dims, strides, box)) return FORGE_ERR_CUDA;
    }
    if (W_NK) {  // w[N, K]: boxes of 64 rows of 64 K-elements (gated: gate rows and up rows; else one or two per CTA)
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)N};
        const uint64_t strides[1] = {(uint64_t)K * 2};
        const uint32_t box[2] = {kBK, 64u};
        if (!encode_tmap_bf16_sw128(&tmap_w, w, 2, dims, strides, box)) return FORGE_ERR_CUDA;
        if (!encode_tmap_bf16_sw128(&tmap_w2, GATED ? w_up : w, 2, dims, strides, box)) return FORGE_ERR_CUDA;
    } else {     // w[K, N]: 64 K-rows of 64 N-elements per box
        const uint64_t dims[2] = {(uint64_t)N, (uint64_t)K};
        const uint64_t strides[1] = {(uint64_t)N * 2};
        const uint32_t box[2] = {64, kBK};
        if (!encode_tmap_bf16_sw128(&tmap_w, w, 2, dims, strides, box)) return FORGE_ERR_CUDA;
        if (!encode_tmap_bf16_sw128(&tmap_w2, GATED ? w_up : w, 2, dims, strides, box)) return FORGE_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)N, (uint64_t)M};
        const uint64_t strides[1] = {(uint64_t)N * 2};
        if (GATED) {  // one epilogue warp's 32 rows x 32 columns, rows of 64 bytes as they lie in its staging buffer
            const uint32_t box[2] = {32, 32};
            if (!encode_tmap_bf16_plain(&tmap_y, y, 2, dims, strides, box)) return FORGE_ERR_CUDA;
        } else {      // one epilogue warp's 32 rows x 64 columns
            const uint32_t box[2] = {64, 32};
            if (!encode_tmap_bf16_sw128(&tmap_y, y, 2, dims, strides, box)) return FORGE_ERR_CUDA;
        }
    }
    int* status = device_status_word();
    if (!status) return FORGE_ERR_CUDA;
    const int sms = sm_count();
    if (sms <= 1) return FORGE_ERR_CUDA;
    auto kernel = linear_pair_kernel<ACT, W_NK, F16, GATED>;
    FORGE_SET_SMEM_ONCE(kernel, L::kAlloc);
    const int tiles = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + BNO - 1) / BNO);
    const int pairs = tiles < sms / 2 ? tiles : sms / 2;
    // the cluster shape is part of the kernel (__cluster_dims__); programmatic stream serialisation as everywhere
    FORGE_CUDA_TRY(launch_pdl(kernel, dim3(2 * pairs), dim3(kThreads), L::kAlloc, s, tmap_x, tmap_w, tmap_w2, tmap_y,
                              static_cast<const uint16_t*>(b), static_cast<const uint16_t*>(residual), M, N, K, status));
    return finish_launch(1);
}

template <bool W_NK, bool F16>
int dispatch_act(int act, const void* x, const void* w, const void* b, const void* r, void* y, int M, int N, int K,
                 cudaStream_t s) {
    switch (act) {
        case FORGE_ACT_GELU_TANH: return launch_pair<FORGE_ACT_GELU_TANH, W_NK, F16>(x, w, b, r, y, M, N, K, s);
        case FORGE_ACT_GELU_ERF: return launch_pair<FORGE_ACT_GELU_ERF, W_NK, F16>(x, w, b, r, y, M, N, K, s);
        case FORGE_ACT_RELU: return launch_pair<FORGE_ACT_RELU, W_NK, F16>(x, w, b, r, y, M, N, K, s);
        case FORGE_ACT_SILU: return launch_pair<FORGE_ACT_SILU, W_NK, F16>(x, w, b, r, y, M, N, K, s);
        default: return launch_pair<FORGE_ACT_NONE, W_NK, F16>(x, w, b, r, y, M, N, K, s);
    }
}

}  // namespace

bool linear_pair_pays(int M, int N, int sms) {
    // Efficiency of a persistent schedule = how full its last round is, times how well the tensor cores are fed:
    // about 0.61 for the one-CTA kernel (operand reads out of L2), about 0.95 for the pair kernel.
    auto fill = [](long long tiles, long long workers) {
        const long long rounds = (tiles + workers - 1) / workers;
        return (double)tiles / (double)(rounds * workers);
    };
    const long long t1 = (long long)((M + 127) / 128) * ((N + 191) / 192);
    const long long t2 = (long long)((M + 255) / 256) * ((N + 255) / 256);
    // with a single row tile the second CTA of every pair would work on padding only
    return sms >= 2 && M > 128 && 0.95 * fill(t2, sms / 2) > 0.61 * fill(t1, sms);
}

int linear_pair_swiglu(const void* x, const void* w_gate, const void* w_up, void* y, int M, int N, int K, int w_layout,
                       cudaStream_t s) {
    return w_layout == FORGE_W_NK
               ? launch_pair<FORGE_ACT_SILU, true, false, true>(x, w_gate, nullptr, nullptr, y, M, N, K, s, w_up)
               : launch_pair<FORGE_ACT_SILU, false, false, true>(x, w_gate, nullptr, nullptr, y, M, N, K, s, w_up);
}

int linear_pair(bool f16, const void* x, const void* w, const void* b, const void* residual, void* y, int M, int N,
                int K, int act, int w_layout, cudaStream_t s) {
    if (f16)
        return w_layout == FORGE_W_NK ? dispatch_act<true, true>(act, x, w, b, residual, y, M, N, K, s)
                                      : dispatch_act<false, true>(act, x, w, b, residual, y, M, N, K, s);
    return w_layout == FORGE_W_NK ? dispatch_act<true, false>(act, x, w, b, residual, y, M, N, K, s)
                                  : dispatch_act<false, false>(act, x, w, b, residual, y, M, N, K, s);
}

}  // namespace forge
