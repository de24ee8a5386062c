// Host-side plumbing of the C ABI: status strings, error bookkeeping, launch counter,
// the device status word, tensor-map encoding and the host-buffer variants.
#include <atomic>
#include <cstring>
#include <mutex>
#include <vector>

#include "forge_common.cuh"
#include "tmap.cuh"

namespace forge {

namespace {
thread_local int tl_last_cuda_error = 0;
std::atomic<unsigned long long> g_launches{0};
__device__ int g_device_status = 0;
}  // namespace

void set_last_cuda_error(cudaError_t e) { tl_last_cuda_error = static_cast<int>(e); }
void count_launch(int n) { g_launches.fetch_add(static_cast<unsigned long long>(n), std::memory_order_relaxed); }

int sm_count() {
    static int cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!cache[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cache[dev] = n;
    }
    return cache[dev];
}

int* device_status_word() {
    // Resolved per device: the symbol has one instance per device that loads the module.
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    static int* cache[64] = {nullptr};
    if (dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_device_status);
        if (e != cudaSuccess) { set_last_cuda_error(e); return nullptr; }
        cache[dev] = static_cast<int*>(p);
    }
    return cache[dev];
}

namespace {
bool encode_tmap_generic(CUtensorMapDataType dtype, CUtensorMapSwizzle swizzle, CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides_bytes, const uint32_t* box) {
    using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !p) {
            set_last_cuda_error(e != cudaSuccess ? e : cudaErrorUnknown);
            return false;
        }
        fn = reinterpret_cast<EncodeFn>(p);
    }
    cuuint64_t gdim[5];
    cuuint64_t gstride[5];
    cuuint32_t gbox[5];
    cuuint32_t estride[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        gbox[i] = box[i];
        estride[i] = 1;
        if (i + 1 < rank) gstride[i] = strides_bytes[i];
    }
    CUresult r = fn(map, dtype, static_cast<cuuint32_t>(rank), const_cast<void*>(base),
                    gdim, gstride, gbox, estride, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error(cudaErrorInvalidValue);
        return false;
    }
    return true;
}
}  // namespace

bool encode_tmap_bf16_sw128(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides_bytes, const uint32_t* box) {
    return encode_tmap_generic(CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, map, base, rank, dims,
                               strides_bytes, box);
}

bool encode_tmap_bf16_plain(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides_bytes, const uint32_t* box) {
    return encode_tmap_generic(CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_NONE, map, base, rank, dims,
                               strides_bytes, box);
}

bool encode_tmap_u8_plain(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                          const uint64_t* strides_bytes, const uint32_t* box) {
    return encode_tmap_generic(CU_TENSOR_MAP_DATA_TYPE_UINT8, CU_TENSOR_MAP_SWIZZLE_NONE, map, base, rank, dims,
                               strides_bytes, box);
}

}  // namespace forge

extern "C" const char* forge_status_string(int status) {
    switch (status) {
        case FORGE_OK: return "FORGE_OK";
        case FORGE_ERR_INVALID_ARG: return "FORGE_ERR_INVALID_ARG";
        case FORGE_ERR_UNSUPPORTED: return "FORGE_ERR_UNSUPPORTED";
        case FORGE_ERR_WORKSPACE: return "FORGE_ERR_WORKSPACE";
        case FORGE_ERR_CUDA: return "FORGE_ERR_CUDA";
        case FORGE_ERR_TIMEOUT: return "FORGE_ERR_TIMEOUT";
        default: return "FORGE_ERR_UNKNOWN";
    }
}

extern "C" int forge_last_cuda_error(void) { return forge::tl_last_cuda_error; }

extern "C" unsigned long long forge_launch_count(void) {
    return forge::g_launches.load(std::memory_order_relaxed);
}

extern "C" int forge_check_status(void* stream) {
    using namespace forge;
    FORGE_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    int* word = device_status_word();
    if (!word) return FORGE_ERR_CUDA;
    int host = 0;
    FORGE_CUDA_TRY(cudaMemcpy(&host, word, sizeof(int), cudaMemcpyDeviceToHost));
    if (host != 0) {
        FORGE_CUDA_TRY(cudaMemset(word, 0, sizeof(int)));
        return FORGE_ERR_TIMEOUT;
    }
    return FORGE_OK;
}

// ------------------------------------------------------------------ host-buffer variants
namespace {
inline size_t up256(size_t n) { return (n + 255) & ~(size_t)255; }

// Two library-owned streams per device for the copies of the host-buffer variants (one per direction) and a
// pool of events to order them against the caller's stream.  A call holds `mu` while it enqueues.
struct CopyLanes {
    std::mutex mu;
    cudaStream_t in = nullptr, out = nullptr;
    std::vector<cudaEvent_t> ev;
};
CopyLanes* copy_lanes(int num_events) {
    static std::mutex table_mu;
    static CopyLanes* table[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(table_mu);
    CopyLanes*& lanes = table[dev];
    if (!lanes) {
        CopyLanes* fresh = new CopyLanes();
        if (cudaStreamCreateWithFlags(&fresh->in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&fresh->out, cudaStreamNonBlocking) != cudaSuccess) {
            delete fresh;
            return nullptr;
        }
        lanes = fresh;
    }
    std::lock_guard<std::mutex> lock2(lanes->mu);
    while ((int)lanes->ev.size() < num_events) {
        cudaEvent_t e;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        lanes->ev.push_back(e);
    }
    return lanes;
}
}  // namespace

extern "C" size_t forge_attn_host_scratch_bytes(int B, int Hq, int Hkv, int Sq, int Skv, int D, int elem_bytes) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Skv <= 0 || D <= 0 || elem_bytes <= 0) return 0;
    const size_t qo = (size_t)B * Hq * Sq * D * elem_bytes;
    const size_t kv = (size_t)B * Hkv * Skv * D * elem_bytes;
    return 2 * up256(qo) + 2 * up256(kv) + up256((size_t)B * 4);
}

static int attn_host_impl(bool f32, const void* q, const void* k, const void* v, void* out,
                          int B, int Hq, int Hkv, int Sq, int Skv, int D,
                          int mask_kind, const int32_t* lens, float scale,
                          void* dev_scratch, size_t dev_scratch_bytes, void* stream) {
    using namespace forge;
    if (!q || !k || !v || !out || !dev_scratch) return FORGE_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Skv <= 0 || D <= 0) return FORGE_ERR_INVALID_ARG;
    if ((mask_kind & FORGE_MASK_PADDING) && !lens) return FORGE_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dev_scratch) & 255u) return FORGE_ERR_INVALID_ARG;
    const int es = f32 ? 4 : 2;
    if (dev_scratch_bytes < forge_attn_host_scratch_bytes(B, Hq, Hkv, Sq, Skv, D, es)) return FORGE_ERR_WORKSPACE;
    const size_t qo = (size_t)B * Hq * Sq * D * es, kv = (size_t)B * Hkv * Skv * D * es;
    char* p = static_cast<char*>(dev_scratch);
    void* dq = p; p += up256(qo);
    void* dk = p; p += up256(kv);
    void* dv = p; p += up256(kv);
    void* dout = p; p += up256(qo);
    int32_t* dlens = reinterpret_cast<int32_t*>(p);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Several batch entries, 16-bit tensors: one entry's copies in, its kernel and its copy out overlap with
    // the neighbours' (the two directions of the host link run at the same time).
    if (!f32 && B >= 2) {
        CopyLanes* lanes = copy_lanes(2 * B + 2);
        if (lanes) {
            std::lock_guard<std::mutex> lock(lanes->mu);
            const size_t qo1 = qo / B, kv1 = kv / B;
            cudaEvent_t fork = lanes->ev[2 * B], join = lanes->ev[2 * B + 1];
            // the library's copy streams start where `stream` is now
            FORGE_CUDA_TRY(cudaEventRecord(fork, s));
            FORGE_CUDA_TRY(cudaStreamWaitEvent(lanes->in, fork, 0));
            FORGE_CUDA_TRY(cudaStreamWaitEvent(lanes->out, fork, 0));
            if (lens) FORGE_CUDA_TRY(cudaMemcpyAsync(dlens, lens, (size_t)B * 4, cudaMemcpyHostToDevice, lanes->in));
            int st = FORGE_OK;
            for (int b = 0; b < B && st == FORGE_OK; ++b) {
                const char* hq = static_cast<const char*>(q) + b * qo1;
                const char* hk = static_cast<const char*>(k) + b * kv1;
                const char* hv = static_cast<const char*>(v) + b * kv1;
                char* dq1 = static_cast<char*>(dq) + b * qo1;
                char* dk1 = static_cast<char*>(dk) + b * kv1;
                char* dv1 = static_cast<char*>(dv) + b * kv1;
                char* do1 = static_cast<char*>(dout) + b * qo1;
                FORGE_CUDA_TRY(cudaMemcpyAsync(dq1, hq, qo1, cudaMemcpyHostToDevice, lanes->in));
                FORGE_CUDA_TRY(cudaMemcpyAsync(dk1, hk, kv1, cudaMemcpyHostToDevice, lanes->in));
                FORGE_CUDA_TRY(cudaMemcpyAsync(dv1, hv, kv1, cudaMemcpyHostToDevice, lanes->in));
                FORGE_CUDA_TRY(cudaEventRecord(lanes->ev[2 * b], lanes->in));
                FORGE_CUDA_TRY(cudaStreamWaitEvent(s, lanes->ev[2 * b], 0));
                st = forge_attn_fused(dq1, dk1, dv1, do1, 1, Hq, Hkv, Sq, Skv, D, mask_kind, lens ? dlens + b : nullptr,
                                      scale, stream);
                if (st != FORGE_OK) break;
                FORGE_CUDA_TRY(cudaEventRecord(lanes->ev[2 * b + 1], s));
                FORGE_CUDA_TRY(cudaStreamWaitEvent(lanes->out, lanes->ev[2 * b + 1], 0));
                FORGE_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(out) + b * qo1, do1, qo1, cudaMemcpyDeviceToHost, lanes->out));
            }
            // `stream` continues after the last copy out (and after everything the copy streams were given)
            FORGE_CUDA_TRY(cudaEventRecord(join, lanes->in));
            FORGE_CUDA_TRY(cudaStreamWaitEvent(s, join, 0));
            FORGE_CUDA_TRY(cudaEventRecord(join, lanes->out));
            FORGE_CUDA_TRY(cudaStreamWaitEvent(s, join, 0));
            return st;
        }
    }
    FORGE_CUDA_TRY(cudaMemcpyAsync(dq, q, qo, cudaMemcpyHostToDevice, s));
    FORGE_CUDA_TRY(cudaMemcpyAsync(dk, k, kv, cudaMemcpyHostToDevice, s));
    FORGE_CUDA_TRY(cudaMemcpyAsync(dv, v, kv, cudaMemcpyHostToDevice, s));
    if (lens) FORGE_CUDA_TRY(cudaMemcpyAsync(dlens, lens, (size_t)B * 4, cudaMemcpyHostToDevice, s));
    int st = f32 ? forge_attn_fused_f32(dq, dk, dv, dout, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens ? dlens : nullptr,
                                        scale, stream)
                 : forge_attn_fused(dq, dk, dv, dout, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens ? dlens : nullptr,
                                    scale, stream);
    if (st != FORGE_OK) return st;
    FORGE_CUDA_TRY(cudaMemcpyAsync(out, dout, qo, cudaMemcpyDeviceToHost, s));
    return FORGE_OK;
}

extern "C" int forge_attn_fused_host(const void* q, const void* k, const void* v, void* out,
                                     int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                     int mask_kind, const int32_t* lens, float scale,
                                     void* dev_scratch, size_t dev_scratch_bytes, void* stream) {
    return attn_host_impl(false, q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, dev_scratch,
                          dev_scratch_bytes, stream);
}

extern "C" int forge_attn_fused_f32_host(const void* q, const void* k, const void* v, void* out,
                                         int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                         int mask_kind, const int32_t* lens, float scale,
                                         void* dev_scratch, size_t dev_scratch_bytes, void* stream) {
    return attn_host_impl(true, q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, dev_scratch,
                          dev_scratch_bytes, stream);
}

extern "C" size_t forge_attn_decode_host_scratch_bytes(int B, int Hq, int Hkv, int Smax, int D, int num_splits) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Smax <= 0 || D <= 0 || num_splits <= 0) return 0;
    const size_t qo = (size_t)B * Hq * D * 2, kv = (size_t)B * Hkv * Smax * D * 2;
    return 2 * up256(qo) + 2 * up256(kv) + up256((size_t)B * 4) +
           up256(forge_attn_decode_workspace_bytes(B, Hq, D, num_splits));
}

extern "C" int forge_attn_decode_splitkv_host(const void* q, const void* k_cache, const void* v_cache, void* out,
                                              int B, int Hq, int Hkv, int Smax, int D,
                                              const int32_t* lens, int num_splits, float scale,
                                              void* dev_scratch, size_t dev_scratch_bytes, void* stream) {
    using namespace forge;
    if (!q || !k_cache || !v_cache || !out || !lens || !dev_scratch) return FORGE_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Smax <= 0 || D <= 0 || num_splits <= 0) return FORGE_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dev_scratch) & 255u) return FORGE_ERR_INVALID_ARG;
    if (dev_scratch_bytes < forge_attn_decode_host_scratch_bytes(B, Hq, Hkv, Smax, D, num_splits))
        return FORGE_ERR_WORKSPACE;
    const size_t qo = (size_t)B * Hq * D * 2, kv = (size_t)B * Hkv * Smax * D * 2;
    const size_t wsb = forge_attn_decode_workspace_bytes(B, Hq, D, num_splits);
    char* p = static_cast<char*>(dev_scratch);
    void* dq = p; p += up256(qo);
    void* dk = p; p += up256(kv);
    void* dv = p; p += up256(kv);
    void* dout = p; p += up256(qo);
    int32_t* dlens = reinterpret_cast<int32_t*>(p); p += up256((size_t)B * 4);
    void* ws = p;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    FORGE_CUDA_TRY(cudaMemcpyAsync(dq, q, qo, cudaMemcpyHostToDevice, s));
    FORGE_CUDA_TRY(cudaMemcpyAsync(dk, k_cache, kv, cudaMemcpyHostToDevice, s));
    FORGE_CUDA_TRY(cudaMemcpyAsync(dv, v_cache, kv, cudaMemcpyHostToDevice, s));
    FORGE_CUDA_TRY(cudaMemcpyAsync(dlens, lens, (size_t)B * 4, cudaMemcpyHostToDevice, s));
    // the scratch is the caller's and may hold anything: the workspace's arrival counters must start at zero
    int st = forge_attn_decode_workspace_init(ws, wsb, stream);
    if (st != FORGE_OK) return st;
    st = forge_attn_decode_splitkv(dq, dk, dv, dout, B, Hq, Hkv, Smax, D, dlens, num_splits, scale, ws, wsb,
                                       stream);
    if (st != FORGE_OK) return st;
    FORGE_CUDA_TRY(cudaMemcpyAsync(out, dout, qo, cudaMemcpyDeviceToHost, s));
    return FORGE_OK;
}

extern "C" size_t forge_linear_host_scratch_bytes(int M, int N, int K) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    return up256((size_t)M * K * 2) + up256((size_t)K * N * 2) + up256((size_t)N * 2) + up256((size_t)M * N * 2);
}

extern "C" int forge_linear_bias_gelu_host(const void* x, const void* w, const void* b, void* y,
                                           int M, int N, int K,
                                           void* dev_scratch, size_t dev_scratch_bytes, void* stream) {
    using namespace forge;
    if (!x || !w || !b || !y || !dev_scratch) return FORGE_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return FORGE_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dev_scratch) & 255u) return FORGE_ERR_INVALID_ARG;
    if (dev_scratch_bytes < forge_linear_host_scratch_bytes(M, N, K)) return FORGE_ERR_WORKSPACE;
    const size_t xb = (size_t)M * K * 2, wb = (size_t)K * N * 2, bb = (size_t)N * 2, yb = (size_t)M * N * 2;
    char* p = static_cast<char*>(dev_scratch);
    void* dx = p; p += up256(xb);
    void* dw = p; p += up256(wb);
    void* db = p; p += up256(bb);
    void* dy = p;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    FORGE_CUDA_TRY(cudaMemcpyAsync(dx, x, xb, cudaMemcpyHostToDevice, s));
    FORGE_CUDA_TRY(cudaMemcpyAsync(dw, w, wb, cudaMemcpyHostToDevice, s));
    FORGE_CUDA_TRY(cudaMemcpyAsync(db, b, bb, cudaMemcpyHostToDevice, s));
    int st = forge_linear_bias_gelu(dx, dw, db, dy, M, N, K, stream);
    if (st != FORGE_OK) return st;
    FORGE_CUDA_TRY(cudaMemcpyAsync(y, dy, yb, cudaMemcpyDeviceToHost, s));
    return FORGE_OK;
}
