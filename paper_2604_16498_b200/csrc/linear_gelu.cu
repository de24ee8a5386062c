// Fused Linear + bias + tanh-GELU (Listing 6 / Eq. 11): Y = gelu_tanh(X W + b) in one kernel.
// The fp32 accumulator lives in tensor memory; bias and activation are applied to it as it is
// read back, before the single rounding to bf16 -- the linear output never reaches memory.
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0    : TMA producer  (X tile 128 x 64, W tile 64 x BN per stage, 128-byte swizzle)
//   warp 1    : tcgen05.mma issuer (one elected lane), owns the TMEM allocation
//   warps 2-9 : epilogue, two warps per TMEM lane quarter, each half of the 64 columns of a block (TMEM -> registers -> +bias -> GELU -> bf16 -> swizzled shared memory -> TMA store)
// Two TMEM accumulators: the epilogue of tile i overlaps the main loop of tile i+1.
// X [M,K] is the K-major A operand; W [K,N] (N contiguous) is the MN-major B operand, so no
// transposed copy of the weights is needed.
// Gated form (SwiGLU, the MLP of the 1B-8B decoder models): Y = silu(X Wg) * (X Wu).  One tile holds
// 128 output columns; its accumulator is 256 columns wide, the gate product in the first half and the
// up product in the second (the B operand of a stage is the gate tile followed by the up tile, one MMA
// of N = 256 per k-step), and the epilogue multiplies the two halves as it reads them back.
// Weight-only int8 form (W8: fp16 activations, int8 weights [N,K] with one fp32 scale per output
// channel, the W-int8/A-fp16 setting of the paper's largest model): 128 x 256 tiles (with one byte per
// weight a 256-column tile stays inside what an SM can pull out of L2 per tensor-core cycle: 32 KB per
// k-step of 512 cycles); the int8 tile of a stage arrives by TMA in the upper half of the stage's B
// operand, eight extra warps (10-17) read all of it into registers, meet at a barrier of their own and
// write the swizzled fp16 operand over it (exact: 1024 + (w ^ 0x80) as fp16 bits, minus 1152); the scale
// is applied to the accumulator in the epilogue, where it factors out of the sum over K.
// Four stages (with a single output staging buffer to make room).  8192 x 8192 x 4096: 511 us (1075 TFLOP/s),
// against 850 us with 192-column tiles, three stages and the int8 tile in a buffer of its own converted
// piece by piece.
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

constexpr int kBM = 128;
constexpr int kBK = 64;
constexpr int kThreads = 320;
constexpr int kEpiThreads = 256;
constexpr int kCvtWarps = 8;      // int8 -> fp16 converter warps of the W8 form
constexpr int kThreadsW8 = kThreads + kCvtWarps * 32;
constexpr int kAccStride = 256;   // TMEM columns between the two accumulators
constexpr int kTmemCols = 512;

template <int BN, int STAGES, bool W8 = false>
struct LinearSmem {
    static constexpr int kABytes = kBM * kBK * 2;        // 16 KB
    static constexpr int kBBytes = kBK * BN * 2;         // 64 rows of K x BN
    // W8: BN rows of 64 int8 weights, which arrive in the upper half of the stage's B operand and are widened in place
    static constexpr int kRawBytes = W8 ? BN * kBK : 0;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kOutBytes = kBM * 128;          // output staging: 128 rows x 64 bf16
    // two buffers; one in the int8 form, whose long k-loops leave the epilogue idle most of the time and whose
    // fourth stage needs the room
    static constexpr int kOutBufs = W8 ? 1 : 2;
    static constexpr int kOutOffset = STAGES * kStageBytes;
    static constexpr int kBarOffset = kOutOffset + kOutBufs * kOutBytes;
    // barriers: full[S], empty[S], tmem_full[2], tmem_empty[2], raw_full[S]; then the TMEM base, then
    // bias[2][BN] and scale[2][BN]
    static constexpr int kBiasOffset = kBarOffset + (3 * STAGES + 4) * 8 + 16;
    static constexpr int kTotal = kBiasOffset + 4 * BN * 4;
    static constexpr int kAlloc = kTotal + 1024;         // slack to align the base to 1024 bytes
};

// 16-bit element helpers: bf16 (F16 = false) or fp16 (F16 = true)
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

// ACT: activation; W_NK: W is stored [N, K] (K-major B operand) instead of [K, N] (MN-major B operand).
// GATED: two weight matrices (tmap_w = gate, tmap_w2 = up), output silu(gate) * up, BN / 2 output columns per tile.
// bias and residual may be null.
// W8: tmap_w2 describes the int8 weights [N,K] (plain layout), `scale` their per-channel factors.
template <int BN, int STAGES, int ACT, bool W_NK, bool GATED, bool F16, bool W8>
__global__ void __launch_bounds__(W8 ? kThreadsW8 : kThreads, 1)
linear_bias_gelu_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                        const __grid_constant__ CUtensorMap tmap_w2,
                        const __grid_constant__ CUtensorMap tmap_y, const uint16_t* __restrict__ bias,
                        const uint16_t* __restrict__ residual, const float* __restrict__ scale, int M, int N, int K,
                        int* __restrict__ status) {
    static_assert(!W8 || (W_NK && F16 && !GATED), "the int8-weight form takes [N,K] weights and fp16 activations");
    using L = LinearSmem<BN, STAGES, W8>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
    uint64_t* empty = full + STAGES;
    uint64_t* tmem_full = empty + STAGES;
    uint64_t* tmem_empty = tmem_full + 2;
    uint64_t* raw_full = tmem_empty + 2;  // W8: the stage's int8 tile has landed
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(raw_full + STAGES);
    volatile uint32_t* epi_gave_up = tmem_base_slot + 1;  // set by an epilogue warp whose wait ran out
    float* s_bias = reinterpret_cast<float*>(smem + L::kBiasOffset);
    float* s_scale = s_bias + 2 * BN;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int BNO = GATED ? BN / 2 : BN;  // output columns per tile
    const int tiles_m = (M + kBM - 1) / kBM, tiles_n = (N + BNO - 1) / BNO;
    const int num_tiles = tiles_m * tiles_n;
    const int kblocks = (K + kBK - 1) / kBK;

    if (threadIdx.x == 0) {
        // W8: a stage is complete when X has landed and the converter warps have written the B operand
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(&full[i], W8 ? 1 + kCvtWarps : 1); mbar_init(&empty[i], 1); mbar_init(&raw_full[i], 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(&tmem_full[i], 1); mbar_init(&tmem_empty[i], kEpiThreads / 32); }
        fence_mbar_init();
        *epi_gave_up = 0;
        prefetch_tmap(&tmap_x);
        prefetch_tmap(&tmap_w);
        if constexpr (GATED) prefetch_tmap(&tmap_w2);
        prefetch_tmap(&tmap_y);
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
    // set-up done: the next kernel may move in as SMs free up; nothing global is touched before the
    // previous kernel has completed
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        if (elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            for (int tile = blockIdx.x; tile < num_tiles && !failed; tile += gridDim.x) {
                const int m0 = (tile / tiles_n) * kBM, n0 = (tile % tiles_n) * BNO;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&empty[stage], phase ^ 1)) { failed = true; break; }
                    uint8_t* sa = smem + stage * L::kStageBytes;
                    uint8_t* sb = sa + L::kABytes;
                    mbar_expect_tx(&full[stage], W8 ? L::kABytes : L::kStageBytes);
                    tma_load_2d(sa, &tmap_x, &full[stage], kb * kBK, m0);
                    if constexpr (W8) {  // BN rows of 64 int8 weights, plain layout, in the upper half of the B operand
                        mbar_expect_tx(&raw_full[stage], L::kRawBytes);
                        tma_load_2d(sb + L::kBBytes - L::kRawBytes, &tmap_w2, &raw_full[stage], kb * kBK, n0);
                    } else if constexpr (W_NK) {  // BN rows of W, 64 K-elements (one swizzle span) each
                        tma_load_2d(sb, &tmap_w, &full[stage], kb * kBK, n0);
                        if constexpr (GATED)  // rows BN/2.. of the operand: the up weights of the same columns
                            tma_load_2d(sb + (BN / 2) * 128, &tmap_w2, &full[stage], kb * kBK, n0);
                    } else {
#pragma unroll
                        for (int c = 0; c < BN / 64; ++c) {
                            if (GATED && c >= BN / 128)
                                tma_load_2d(sb + c * (kBK * 128), &tmap_w2, &full[stage], n0 + (c - BN / 128) * 64, kb * kBK);
                            else
                                tma_load_2d(sb + c * (kBK * 128), &tmap_w, &full[stage], n0 + c * 64, kb * kBK);
                        }
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc = F16 ? make_idesc_f16(kBM, BN, /*a_mn_major=*/false, /*b_mn_major=*/!W_NK)
                                           : make_idesc_bf16(kBM, BN, /*a_mn_major=*/false, /*b_mn_major=*/!W_NK);
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            for (int tile = blockIdx.x; tile < num_tiles && !failed; tile += gridDim.x, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!mbar_wait(&tmem_empty[acc], acc_phase ^ 1)) { failed = true; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * kAccStride;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&full[stage], phase)) { failed = true; break; }
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
                    const uint32_t sb = sa + L::kABytes;
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        // A: 16 K-elements = 32 bytes further along the 128-byte swizzled row
                        const uint64_t a_desc = make_smem_desc(sa + k * 32, 16, 1024);
                        // B: 16 K-rows = two 1024-byte groups further; 64-column chunks are kBK*128 bytes apart
                        // [N,K] weights: K-major like A (32 bytes per k-step inside the swizzled row)
                        const uint64_t b_desc = W_NK ? make_smem_desc(sb + k * 32, 16, 1024)
                                                     : make_smem_desc(sb + k * 2048, kBK * 128, 1024);
                        mma_ss(d_tmem, a_desc, b_desc, idesc, (kb | k) != 0);
                    }
                    mma_commit(&empty[stage]);  // the stage is free once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (failed) break;
                mma_commit(&tmem_full[acc]);
            }
        }
    } else if (W8 && warp >= 10) {
        // ------------------------------------------------------------------ int8 -> fp16 converters
        // Thread t of the converter warps takes 16-byte pieces t, t + 256, ... of the stage's int8 tile: piece q holds
        // weights 16 (q % 4) .. +15 of row q / 4, which become 16-byte chunks 2 (q % 4) and 2 (q % 4) + 1 of
        // that row's 128-byte line of the K-major, 128-byte-swizzled B operand.
        const int ctid = (warp - 10) * 32 + lane;
        int stage = 0;
        uint32_t phase = 0;
        for (int tile = blockIdx.x; tile < num_tiles && !failed; tile += gridDim.x) {
            for (int kb = 0; kb < kblocks; ++kb) {
                if (!warp_wait(&raw_full[stage], phase)) { failed = true; break; }
                uint8_t* sb = smem + stage * L::kStageBytes + L::kABytes;
                const uint8_t* raw = sb + L::kBBytes - L::kRawBytes;
                constexpr int kPieces = BN * 4 / (kCvtWarps * 32);  // 16-byte pieces per thread
                uint4 in[kPieces];
#pragma unroll
                for (int i = 0; i < kPieces; ++i) in[i] = *reinterpret_cast<const uint4*>(raw + (i * (kCvtWarps * 32) + ctid) * 16);
                // the fp16 rows of the upper half overwrite the int8 tile: every piece must have been read first
                asm volatile("bar.sync 2, %0;" ::"n"(kCvtWarps * 32) : "memory");
#pragma unroll
                for (int i = 0; i < kPieces; ++i) {
                    const int q = i * (kCvtWarps * 32) + ctid, n = q >> 2, part = q & 3;
                    const uint32_t wds[4] = {in[i].x ^ 0x80808080u, in[i].y ^ 0x80808080u, in[i].z ^ 0x80808080u, in[i].w ^ 0x80808080u};
                    uint32_t o[8];
                    const __half2 off = __floats2half2_rn(1152.f, 1152.f);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // bytes (u, 0x64) read as fp16 are 1024 + u; u = w + 128
                        uint32_t lo = __byte_perm(wds[j], 0x64646464u, 0x4140), hi = __byte_perm(wds[j], 0x64646464u, 0x4342);
                        __half2 hlo = __hsub2(*reinterpret_cast<__half2*>(&lo), off);
                        __half2 hhi = __hsub2(*reinterpret_cast<__half2*>(&hi), off);
                        o[2 * j] = *reinterpret_cast<uint32_t*>(&hlo);
                        o[2 * j + 1] = *reinterpret_cast<uint32_t*>(&hhi);
                    }
                    uint8_t* line = sb + n * 128;
                    *reinterpret_cast<uint4*>(line + (((2 * part) ^ (n & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                    *reinterpret_cast<uint4*>(line + (((2 * part + 1) ^ (n & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
                }
                fence_proxy_async_smem();  // the tensor core reads what these threads wrote
                __syncwarp();
                if (lane == 0) mbar_arrive(&full[stage]);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else {
        const int quarter = warp & 3;            // TMEM lane quarter this warp may access
        const int etid = (warp - 2) * 32 + lane; // 0..255
        const int chalf = (warp - 2) >> 2;       // which 32 of a block's 64 columns this warp handles
        int it = 0;
        int out_blocks = 0;  // 64-column blocks stored so far (selects the staging buffer)
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
            const int m0 = (tile / tiles_n) * kBM, n0 = (tile % tiles_n) * BNO;
            const int acc = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1;
            float* bias_s = s_bias + acc * BN;
            float* scale_s = s_scale + acc * BN;
            for (int i = etid; i < BNO; i += kEpiThreads) {
                bias_s[i] = (bias != nullptr && n0 + i < N) ? widen16<F16>(bias[n0 + i]) : 0.f;
                if constexpr (W8) scale_s[i] = (n0 + i < N) ? scale[n0 + i] : 0.f;
            }
            // The accumulator is complete.  Whether to go on is decided for the whole epilogue group: a warp
            // whose wait ran out says so in shared memory before the barrier, and all eight warps read the
            // flag after it, so either all of them enter the block loop below (whose barriers need all of
            // them) or all leave.
            if (!warp_wait(&tmem_full[acc], acc_phase) && lane == 0) *epi_gave_up = 1;
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");  // also publishes bias_s / scale_s
            if (*epi_gave_up) { failed = true; break; }
            tc_fence_after_sync();
            const int row = quarter * 32 + lane;  // row of the tile = TMEM lane
            const uint32_t taddr = tmem_base + acc * kAccStride + (static_cast<uint32_t>(quarter * 32) << 16);
            // 64 output columns at a time: registers -> bf16 -> swizzled staging buffer -> one TMA store.
            // Two staging buffers: the store of one block drains while the next block is computed.
#pragma unroll 1
            for (int blk = 0; blk < BNO / 64; ++blk, ++out_blocks) {
                uint8_t* stage_out = smem + L::kOutOffset + (out_blocks % L::kOutBufs) * L::kOutBytes;
                uint32_t r[32];
                tmem_ld_x32(taddr + blk * 64 + chalf * 32, r);
                if constexpr (GATED) {  // silu(gate) * up, the up product sits BN / 2 columns further
                    uint32_t r2[32];
                    tmem_ld_x32(taddr + BN / 2 + blk * 64 + chalf * 32, r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        r[i] = __float_as_uint(activate<FORGE_ACT_SILU>(__uint_as_float(r[i])) * __uint_as_float(r2[i]));
                }
                tmem_ld_wait();
                // the store that last used this buffer (two blocks ago with two buffers) has finished reading it
                if (etid == 0) tma_store_wait_read<L::kOutBufs - 1>();
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
#pragma unroll
                for (int c = 0; c < 4; ++c) {  // 16-byte chunk chalf*4 + c of the row's 128-byte line
                    uint32_t w[4];
                    // residual[m, n .. n+7] (mm+add pattern): 16 bytes of this thread's output row
                    uint4 res = make_uint4(0, 0, 0, 0);
                    const int gcol = n0 + blk * 64 + chalf * 32 + c * 8;
                    if (residual != nullptr && m0 + row < M && gcol < N)
                        res = *reinterpret_cast<const uint4*>(residual + (size_t)(m0 + row) * N + gcol);
                    const uint32_t rw[4] = {res.x, res.y, res.z, res.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int col = c * 8 + 2 * i;
                        const int bc = blk * 64 + chalf * 32 + col;
                        float z0 = __uint_as_float(r[col]), z1 = __uint_as_float(r[col + 1]);
                        if constexpr (W8) { z0 *= scale_s[bc]; z1 *= scale_s[bc + 1]; }
                        z0 += bias_s[bc];
                        z1 += bias_s[bc + 1];
                        w[i] = pack16<F16>(activate<GATED ? FORGE_ACT_NONE : ACT>(z0) + widen16<F16>(static_cast<uint16_t>(rw[i] & 0xffffu)),
                                           activate<GATED ? FORGE_ACT_NONE : ACT>(z1) + widen16<F16>(static_cast<uint16_t>(rw[i] >> 16)));
                    }
                    *reinterpret_cast<uint4*>(stage_out + row * 128 + (((chalf * 4 + c) ^ (row & 7)) << 4)) =
                        make_uint4(w[0], w[1], w[2], w[3]);
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                if (etid == 0) {
                    // rows >= M and columns >= N are clipped by the TMA unit
                    tma_store_2d(&tmap_y, stage_out, n0 + blk * 64, m0);
                    tma_store_commit();
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        }
        if (etid == 0) tma_store_wait_all<0>();  // every output tile has left shared memory and is written
    }

    if (failed) {
        atomicExch(status, 1);
        // give copies and MMAs that are still in flight time to land before TMEM and smem go away
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <int BN, int STAGES, int ACT, bool W_NK, bool GATED = false, bool F16 = false, bool W8 = false>
int launch_linear(const void* x, const void* w, const void* b, const void* residual, void* y, int M, int N, int K,
                  cudaStream_t s, const void* w_up = nullptr, const float* scale = nullptr) {
    using L = LinearSmem<BN, STAGES, W8>;
    constexpr int BNO = GATED ? BN / 2 : BN;
    CUtensorMap tmap_x, tmap_w, tmap_w2, tmap_y;
    {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
        const uint64_t strides[1] = {(uint64_t)K * 2};
        const uint32_t box[2] = {kBK, kBM};
        if (!encode_tmap_bf16_sw128(&tmap_x, x, 2, dims, strides, box)) return FORGE_ERR_CUDA;
    }
    if (W8) {    // int8 w[N, K]: BN rows of 64 bytes per box, plain layout; no 16-bit weight map is used
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)N};
        const uint64_t strides[1] = {(uint64_t)K};
        const uint32_t box[2] = {kBK, BNO};
        if (!encode_tmap_u8_plain(&tmap_w2, w, 2, dims, strides, box)) return FORGE_ERR_CUDA;
        tmap_w = tmap_w2;
    } else if (W_NK) {  // w[N, K]: rows of 64 K-elements
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)N};
        const uint64_t strides[1] = {(uint64_t)K * 2};
        const uint32_t box[2] = {kBK, BNO};
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
        const uint32_t box[2] = {64, kBM};
        if (!encode_tmap_bf16_sw128(&tmap_y, y, 2, dims, strides, box)) return FORGE_ERR_CUDA;
    }
    int* status = device_status_word();
    if (!status) return FORGE_ERR_CUDA;
    const int sms = sm_count();
    if (sms <= 0) return FORGE_ERR_CUDA;
    auto kernel = linear_bias_gelu_kernel<BN, STAGES, ACT, W_NK, GATED, F16, W8>;
    FORGE_SET_SMEM_ONCE(kernel, L::kAlloc);
    const int tiles = ((M + kBM - 1) / kBM) * ((N + BNO - 1) / BNO);
    const int grid = tiles < sms ? tiles : sms;
    FORGE_CUDA_TRY(launch_pdl(kernel, dim3(grid), dim3(W8 ? kThreadsW8 : kThreads), L::kAlloc, s, tmap_x, tmap_w, tmap_w2,
                              tmap_y, static_cast<const uint16_t*>(b), static_cast<const uint16_t*>(residual), scale,
                              M, N, K, status));
    return finish_launch(1);
}

template <int ACT, bool F16>
int launch_layout(int w_layout, const void* x, const void* w, const void* b, const void* r, void* y, int M, int N,
                  int K, cudaStream_t s) {
    // This kernel gets the problems with a single row tile (M <= 128): they stream W once and are bound by HBM, so
    // what counts is how many SMs pull on it.  When 192-column tiles would leave many SMs without one (and W is
    // large enough for that to matter: small problems are bound by latency, which more and narrower tiles only
    // add to), narrower tiles with deeper rings spread the same bytes over more of them: the widest of 192, 128
    // and 64 columns that gives at least three quarters of the SMs a tile, else 64.
    const int sms = sm_count();
    const long long w_bytes = 2LL * N * K;
    if ((N + 191) / 192 < (3 * sms) / 4 && w_bytes >= (16LL << 20)) {
        if ((N + 127) / 128 >= (3 * sms) / 4)
            return w_layout == FORGE_W_NK ? launch_linear<128, 5, ACT, true, false, F16>(x, w, b, r, y, M, N, K, s)
                                          : launch_linear<128, 5, ACT, false, false, F16>(x, w, b, r, y, M, N, K, s);
        return w_layout == FORGE_W_NK ? launch_linear<64, 8, ACT, true, false, F16>(x, w, b, r, y, M, N, K, s)
                                      : launch_linear<64, 8, ACT, false, false, F16>(x, w, b, r, y, M, N, K, s);
    }
    return w_layout == FORGE_W_NK ? launch_linear<192, 4, ACT, true, false, F16>(x, w, b, r, y, M, N, K, s)
                                  : launch_linear<192, 4, ACT, false, false, F16>(x, w, b, r, y, M, N, K, s);
}

template <bool F16>
int linear_act_impl(const void* x, const void* w, const void* b, const void* residual, void* y,
                    int M, int N, int K, int act, int w_layout, void* stream) {
    if (!x || !w || !y) return FORGE_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return FORGE_ERR_INVALID_ARG;
    if (act < FORGE_ACT_GELU_TANH || act > FORGE_ACT_NONE) return FORGE_ERR_INVALID_ARG;
    if (w_layout != FORGE_W_KN && w_layout != FORGE_W_NK) return FORGE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || (b && !aligned16(b)) || (residual && !aligned16(residual)))
        return FORGE_ERR_INVALID_ARG;
    if ((K % 8) != 0 || (N % 8) != 0) return FORGE_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // large outputs run on CTA pairs (see linear_pair.cu); shapes with few tiles stay on the one-CTA kernel
    if (linear_pair_pays(M, N, sm_count())) return linear_pair(F16, x, w, b, residual, y, M, N, K, act, w_layout, s);
    switch (act) {
        case FORGE_ACT_GELU_TANH: return launch_layout<FORGE_ACT_GELU_TANH, F16>(w_layout, x, w, b, residual, y, M, N, K, s);
        case FORGE_ACT_GELU_ERF: return launch_layout<FORGE_ACT_GELU_ERF, F16>(w_layout, x, w, b, residual, y, M, N, K, s);
        case FORGE_ACT_RELU: return launch_layout<FORGE_ACT_RELU, F16>(w_layout, x, w, b, residual, y, M, N, K, s);
        case FORGE_ACT_SILU: return launch_layout<FORGE_ACT_SILU, F16>(w_layout, x, w, b, residual, y, M, N, K, s);
        default: return launch_layout<FORGE_ACT_NONE, F16>(w_layout, x, w, b, residual, y, M, N, K, s);
    }
}

}  // namespace
}  // namespace forge

extern "C" int forge_linear_act(const void* x, const void* w, const void* b, const void* residual, void* y,
                                int M, int N, int K, int act, int w_layout, void* stream) {
    return forge::linear_act_impl<false>(x, w, b, residual, y, M, N, K, act, w_layout, stream);
}

extern "C" int forge_linear_act_f16(const void* x, const void* w, const void* b, const void* residual, void* y,
                                    int M, int N, int K, int act, int w_layout, void* stream) {
    return forge::linear_act_impl<true>(x, w, b, residual, y, M, N, K, act, w_layout, stream);
}

extern "C" int forge_linear_bias_gelu(const void* x, const void* w, const void* b, void* y,
                                      int M, int N, int K, void* stream) {
    if (!b) return FORGE_ERR_INVALID_ARG;
    return forge_linear_act(x, w, b, nullptr, y, M, N, K, FORGE_ACT_GELU_TANH, FORGE_W_KN, stream);
}

extern "C" int forge_linear_swiglu(const void* x, const void* w_gate, const void* w_up, void* y,
                                   int M, int N, int K, int w_layout, void* stream) {
    using namespace forge;
    if (!x || !w_gate || !w_up || !y) return FORGE_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return FORGE_ERR_INVALID_ARG;
    if (w_layout != FORGE_W_KN && w_layout != FORGE_W_NK) return FORGE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w_gate) || !aligned16(w_up) || !aligned16(y)) return FORGE_ERR_INVALID_ARG;
    if ((K % 8) != 0 || (N % 8) != 0) return FORGE_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // more than one row tile: CTA pairs (see linear_pair.cu)
    if (M > 128 && sm_count() >= 2) return linear_pair_swiglu(x, w_gate, w_up, y, M, N, K, w_layout, s);
    return w_layout == FORGE_W_NK
               ? launch_linear<256, 3, FORGE_ACT_SILU, true, true>(x, w_gate, nullptr, nullptr, y, M, N, K, s, w_up)
               : launch_linear<256, 3, FORGE_ACT_SILU, false, true>(x, w_gate, nullptr, nullptr, y, M, N, K, s, w_up);
}

extern "C" int forge_linear_act_w8a16(const void* x, const void* w_int8, const float* scale, const void* b,
                                      const void* residual, void* y, int M, int N, int K, int act, void* stream) {
    using namespace forge;
    if (!x || !w_int8 || !scale || !y) return FORGE_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return FORGE_ERR_INVALID_ARG;
    if (act < FORGE_ACT_GELU_TANH || act > FORGE_ACT_NONE) return FORGE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w_int8) || !aligned16(y) || (b && !aligned16(b)) || (residual && !aligned16(residual)) ||
        (reinterpret_cast<uintptr_t>(scale) & 3u))
        return FORGE_ERR_INVALID_ARG;
    if ((K % 16) != 0 || (N % 8) != 0) return FORGE_ERR_UNSUPPORTED;  // 16-byte rows of int8 weights and of fp16 outputs
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (act) {
        case FORGE_ACT_GELU_TANH: return launch_linear<256, 4, FORGE_ACT_GELU_TANH, true, false, true, true>(x, w_int8, b, residual, y, M, N, K, s, nullptr, scale);
        case FORGE_ACT_GELU_ERF: return launch_linear<256, 4, FORGE_ACT_GELU_ERF, true, false, true, true>(x, w_int8, b, residual, y, M, N, K, s, nullptr, scale);
        case FORGE_ACT_RELU: return launch_linear<256, 4, FORGE_ACT_RELU, true, false, true, true>(x, w_int8, b, residual, y, M, N, K, s, nullptr, scale);
        case FORGE_ACT_SILU: return launch_linear<256, 4, FORGE_ACT_SILU, true, false, true, true>(x, w_int8, b, residual, y, M, N, K, s, nullptr, scale);
        default: return launch_linear<256, 4, FORGE_ACT_NONE, true, false, true, true>(x, w_int8, b, residual, y, M, N, K, s, nullptr, scale);
    }
}
