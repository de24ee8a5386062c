/*
 * forge.h -- C ABI of the B200 (sm_100a) library for the fused patterns that the
 * attention-fusion and operator-fusion passes of the FORGE-UGC compiler produce:
 *
 *   - fused scaled-dot-product attention: the chain  Q.K^T -> scale -> [mask] ->
 *     softmax -> .V  collapsed into one operator (Section 4.3 "Pass 4: Attention
 *     Fusion", Eq. 8 and Eq. 9), with grouped-query heads and a split-KV decode
 *     variant;
 *   - fused Linear + bias + GELU: matmul, element-wise bias add and activation in
 *     one dispatch, the linear output never materialised (Section 4.3 "Pass 5:
 *     Operator Fusion", Listing 6 and Eq. 11).
 *
 * Conventions shared by every entry point
 *   - Unless a parameter says HOST, pointers are DEVICE pointers owned by the
 *     caller.  The library never frees or keeps them and allocates no device
 *     memory.  Pointers must be 16-byte aligned.
 *   - Tensors are dense, row-major, last index fastest:
 *       q, out : [B, Hq, Sq, D]        k, v : [B, Hkv, Skv, D]        lens : int32 [B]
 *   - Query head h reads KV head h / (Hq / Hkv)  (consecutive grouping).
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream).  No entry point synchronises unless it says so.
 *   - Arguments are validated on the host before anything is launched.  The return
 *     value is a forge_status; nothing throws.
 *   - mask_kind: FORGE_MASK_NONE, FORGE_MASK_CAUSAL, FORGE_MASK_PADDING (key j of
 *     sequence b is valid iff j < lens[b]) or FORGE_MASK_CAUSAL_PADDING.  A masked
 *     key gets probability exactly 0.  Causal alignment for Sq != Skv is
 *     bottom-right: query i sees keys j <= i + (Skv - Sq).  lens lives on the
 *     device, so it cannot be checked on the host: kernels clamp lens[b] to
 *     [0, Skv]; a query row with no visible key yields zeros.
 *   - Dropout, which the matched chain may contain, is the identity at inference
 *     and is not implemented.
 */
#ifndef FORGE_H_
#define FORGE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum forge_status {
    FORGE_OK = 0,
    FORGE_ERR_INVALID_ARG = 1, /* NULL pointer, non-positive size, Hq % Hkv != 0, misaligned pointer, lens missing */
    FORGE_ERR_UNSUPPORTED = 2, /* valid request with no kernel: D not in {64,128}, row stride not a multiple of 16 bytes, ... */
    FORGE_ERR_WORKSPACE = 3,   /* workspace too small */
    FORGE_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; see forge_last_cuda_error() */
    FORGE_ERR_TIMEOUT = 5      /* a bounded wait inside a kernel expired; reported by forge_check_status() */
} forge_status;

enum {
    FORGE_MASK_NONE = 0,
    FORGE_MASK_CAUSAL = 1,
    FORGE_MASK_PADDING = 2,
    FORGE_MASK_CAUSAL_PADDING = 3
};

/*
 * Fused attention, bf16 in / fp32 accumulate / bf16 out:
 *     out[b,h,i,:] = sum_j softmax_j(scale * q[b,h,i,:].k[b,h/G,j,:] over visible j) * v[b,h/G,j,:]
 * (Eq. 9 with the optional scale and mask nodes of Eq. 8 folded in; scores and
 * probabilities never reach global memory).  D: any multiple of 8 up to 256 (sizes other than 64, 128 and
 * 256 run on the next larger kernel: the TMA unit pads the rows with zeros on the fly; sizes above 128 run
 * on a kernel of their own with one query tile per CTA).  `lens` may be
 * NULL unless mask_kind has the padding bit.  scale must be >= 0 (FORGE_ERR_UNSUPPORTED otherwise: the
 * kernel takes the running maximum on unscaled scores; forge_attn_fused_f32 accepts any sign).  Padded
 * K and V rows (beyond lens[b]) may hold anything, including NaN and Inf: they never reach the result.
 * Tensor-core path (tcgen05, TMEM accumulators, TMA-staged K/V).
 */
int forge_attn_fused(const void* q, const void* k, const void* v, void* out,
                     int B, int Hq, int Hkv, int Sq, int Skv, int D,
                     int mask_kind, const int32_t* lens, float scale, void* stream);

/*
 * Same operator, same kernel, with fp16 tensors in and out (fp32 accumulate; the
 * probabilities are rounded to fp16 before the product with V).  fp16 is the
 * inference precision of the paper's evaluation (Section 5.1, model table).
 * Same arguments, limits and errors as forge_attn_fused.  |scale * q.k| beyond
 * what fp32 holds is the caller's concern; outputs are convex combinations of V
 * rows and cannot overflow fp16 unless V does.
 */
int forge_attn_fused_f16(const void* q, const void* k, const void* v, void* out,
                         int B, int Hq, int Hkv, int Sq, int Skv, int D,
                         int mask_kind, const int32_t* lens, float scale, void* stream);

/*
 * forge_attn_fused on tensors that are views of larger buffers: the same operator (Eq. 9), same kernel,
 * bf16, but q, k, v and out are addressed through element strides {batch, head, row} given by the caller
 * (x_strides[0..2]); the D elements of a row are contiguous.  This is what lets the operator read the
 * output of a fused QKV projection ([tokens, (Hq + 2 Hkv) D], i.e. [B, S, heads, D]) and write what the
 * output projection reads ([tokens, Hq D]) without any copy in between: the dense layout of
 * forge_attn_fused is the special case {H S D, S D, D}.  Every stride must be positive and a multiple
 * of 8 elements (rows start on 16-byte boundaries), the row stride at least D; FORGE_ERR_INVALID_ARG /
 * FORGE_ERR_UNSUPPORTED otherwise.  Everything else as forge_attn_fused.
 */
int forge_attn_fused_strided(const void* q, const void* k, const void* v, void* out,
                             int B, int Hq, int Hkv, int Sq, int Skv, int D,
                             const int64_t* q_strides, const int64_t* k_strides, const int64_t* v_strides,
                             const int64_t* out_strides, int mask_kind, const int32_t* lens, float scale,
                             void* stream);

/*
 * forge_attn_fused with the optional mask node of the fused pattern (Eq. 8) given as a
 * tensor: bias [B, bias_heads, Sq, Skv] fp32 on the device (16-byte aligned, contiguous),
 * bias_heads = 1 (shared by all query heads) or Hq, is added to the scaled scores before
 * the softmax:  softmax_j(scale * q.k_j + bias[b, h, i, j]).  An entry of -infinity
 * excludes the key; a row whose keys are all excluded gives zeros.  Finite entries are
 * arbitrary (relative-position or ALiBi-style biases), but a "large negative" stand-in
 * for -infinity must stay finite after division by scale.  mask_kind / lens apply on top.
 * bf16 q, k, v, out as in forge_attn_fused, D up to 128.  scale must be > 0 (FORGE_ERR_UNSUPPORTED
 * otherwise); other errors as forge_attn_fused.
 */
int forge_attn_fused_bias(const void* q, const void* k, const void* v, void* out,
                          int B, int Hq, int Hkv, int Sq, int Skv, int D,
                          int mask_kind, const int32_t* lens, const float* bias, int bias_heads,
                          float scale, void* stream);

/*
 * Same operator with fp32 tensors in and out (fp32 FMA arithmetic, no reduced
 * precision inside).  D must be 64 or 128.
 */
int forge_attn_fused_f32(const void* q, const void* k, const void* v, void* out,
                         int B, int Hq, int Hkv, int Sq, int Skv, int D,
                         int mask_kind, const int32_t* lens, float scale, void* stream);

/*
 * Decode step of the same operator (Eq. 9 with one query row per head) over a KV
 * cache, split along the cached sequence, with the combine step in the same kernel:
 *     q, out : [B, Hq, D] bf16       k_cache, v_cache : [B, Hkv, Smax, D] bf16
 * Sequence b attends rows 0 .. lens[b]-1 of its cache (lens[b] clamped to
 * [0, Smax]; 0 gives zeros).  Rows at and beyond lens[b] may hold anything.
 *
 * Split rule.  Every sequence is cut into pieces of c 16-row blocks, counted from its
 * start (the last piece may be shorter), with one c for the whole call, chosen on the
 * device from lens: the smallest c with
 *     c >= ceil(blocks of all sequences and kv heads / workers)   (workers = 8 per SM)
 *     c >= ceil(blocks of the longest sequence / num_splits),
 * raised by up to a factor of about two if that leaves no more pieces than workers.
 * So num_splits is the largest number of pieces any sequence is cut into, and in a
 * batch that fills the GPU every worker streams one piece of the same length.  Each
 * piece produces a partial (running max, running sum, unnormalised output, fp32) in
 * `workspace`; the worker that completes the last piece of a (batch, kv head) merges
 * its partials and writes the output rows.  A sequence with a single piece never
 * touches the workspace.  The result does not depend on num_splits beyond rounding.
 *
 * workspace: at least forge_attn_decode_workspace_bytes(...) bytes, 16-byte aligned.
 * It starts with one arrival counter per (batch, kv head), which must be ZERO when a
 * call starts: clear a new workspace once with forge_attn_decode_workspace_init (or
 * any memset); every call that completes leaves the counters at zero, so the same
 * workspace can be passed again and again.  The counters take the first
 * max(1088 KiB, 68 * B * Hq bytes): all shapes with B * Hq <= 16384 share that region, so
 * a workspace cleared once also serves later calls of other such shapes; after a call
 * with a larger B * Hq, or one that ended in FORGE_ERR_TIMEOUT, clear it again.  The
 * rest needs no initialisation.  Two calls that may overlap on the GPU must not share
 * a workspace.
 * 1 <= num_splits <= 256 (FORGE_ERR_UNSUPPORTED beyond); D any multiple of 8 up to 128; Hq / Hkv
 * must be between 1 and 8.  A piece is streamed by one warp, and a GPU runs seven such warps
 * per SM: with few (batch, kv head) pairs, allow about 7 * SMs / (B * Hkv) pieces per sequence
 * (a single sequence with 8 kv heads: 128 or more) or most of the GPU idles.
 */
int forge_attn_decode_splitkv(const void* q, const void* k_cache, const void* v_cache, void* out,
                              int B, int Hq, int Hkv, int Smax, int D,
                              const int32_t* lens, int num_splits, float scale,
                              void* workspace, size_t workspace_bytes, void* stream);

/* The same decode step with fp16 q, caches and out (the paper's inference precision); everything else,
 * including the workspace size, as forge_attn_decode_splitkv. */
int forge_attn_decode_splitkv_f16(const void* q, const void* k_cache, const void* v_cache, void* out,
                                  int B, int Hq, int Hkv, int Smax, int D,
                                  const int32_t* lens, int num_splits, float scale,
                                  void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of workspace forge_attn_decode_splitkv needs; 0 for invalid arguments. */
size_t forge_attn_decode_workspace_bytes(int B, int Hq, int D, int num_splits);

/* Clears a decode workspace (a memset enqueued on `stream`): needed once after allocation, and after a
 * call that ended in FORGE_ERR_TIMEOUT.  Belongs to the split-KV decode step above. */
int forge_attn_decode_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * forge_attn_decode_splitkv for callers that cannot provide a workspace because they cannot
 * allocate device memory at all (the paper has no counterpart to this entry point; it exists
 * for deployment reasons only).  Typical cases: a serving process whose device-memory plan is
 * frozen once it has started, a plugin inside a host runtime that owns the allocator, a latency
 * path that must avoid the device-wide synchronisation cudaMalloc implies.
 *
 * The split partials go to a fixed array of FORGE_DECODE_STATIC_SCRATCH_BYTES that is compiled
 * into the library's device image; every GPU that loads the library holds that much memory until
 * the process exits.  The call itself allocates and frees nothing, on the host or on the device.
 * Inputs, `out` and `lens` are still the caller's device buffers, with the same meaning, layout
 * and limits as forge_attn_decode_splitkv, and the result is the same.
 *
 *   - Problems whose partials do not fit, i.e. forge_attn_decode_workspace_bytes(B, Hq, D,
 *     num_splits) > FORGE_DECODE_STATIC_SCRATCH_BYTES, are refused with FORGE_ERR_WORKSPACE and
 *     nothing is launched (B=16, Hq=32, D=128, 16 splits needs 4.2 MiB).
 *   - The first call on each device looks up the array's device address (the device must be
 *     current).  Make that first call outside any stream capture; later calls do no set-up.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left
 *     there.  The arrival counters at its start are zero when the library is loaded and every
 *     completed call puts them back to zero; the partial slots are overwritten before they are
 *     read.  So nothing needs clearing between calls, but two calls that may run at the same time
 *     on one GPU (streams or host threads of this process on the same device) race on the array
 *     and give wrong results: serialise them, or use forge_attn_decode_splitkv with one workspace
 *     per concurrent call.  Other processes have their own copy of the array.  A call that ended
 *     in FORGE_ERR_TIMEOUT may leave counters behind; this entry point then stays unusable on
 *     that device for the rest of the process.
 *   - A slot holds (D <= 64 ? 64 : 128) + 2 floats per (batch, head, piece).
 */
#define FORGE_DECODE_STATIC_SCRATCH_BYTES (8u << 20)
int forge_attn_decode_splitkv_static(const void* q, const void* k_cache, const void* v_cache, void* out,
                                     int B, int Hq, int Hkv, int Smax, int D,
                                     const int32_t* lens, int num_splits, float scale, void* stream);

/*
 * Fused Linear + bias + tanh-GELU (Listing 6 / Eq. 11):
 *     y[m,n] = gelu_tanh(b[n] + sum_k x[m,k] * w[k,n]),
 *     gelu_tanh(z) = 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3)))
 * x [M,K], w [K,N] (GPT-2 c_fc layout), b [N], y [M,N]; bf16 in and out, fp32
 * accumulation, bias and activation applied to the fp32 accumulator before the
 * single rounding to bf16.  K and N must be multiples of 8 (16-byte rows).
 * Tensor-core path (tcgen05, TMEM accumulators, TMA-staged operands).
 */
int forge_linear_bias_gelu(const void* x, const void* w, const void* b, void* y,
                           int M, int N, int K, void* stream);

/*
 * The other patterns of the operator-fusion pass (Section 4.3 "Pass 5": linear+relu, linear+gelu,
 * linear+silu, and mm+add, a residual addition after a raw matrix multiply), on the same kernel:
 *     y[m,n] = act(b[n] + sum_k x[m,k] * W(k,n)) + residual[m,n]
 * act: FORGE_ACT_GELU_TANH, FORGE_ACT_GELU_ERF (0.5 z (1 + erf(z / sqrt 2))), FORGE_ACT_RELU,
 * FORGE_ACT_SILU (z / (1 + exp(-z))) or FORGE_ACT_NONE.  w_layout: FORGE_W_KN = w stored [K,N] (as in
 * forge_linear_bias_gelu), FORGE_W_NK = w stored [N,K], the [out,in] layout of the listing's Linear.
 * b ([N]) and residual ([M,N], bf16) may be NULL.  Same shape limits as forge_linear_bias_gelu.
 */
enum { FORGE_ACT_GELU_TANH = 0, FORGE_ACT_GELU_ERF = 1, FORGE_ACT_RELU = 2, FORGE_ACT_SILU = 3, FORGE_ACT_NONE = 4 };
enum { FORGE_W_KN = 0, FORGE_W_NK = 1 };
int forge_linear_act(const void* x, const void* w, const void* b, const void* residual, void* y,
                     int M, int N, int K, int act, int w_layout, void* stream);

/* forge_linear_act with fp16 x, w, b, residual and y (fp32 accumulation; same arguments and limits). */
int forge_linear_act_f16(const void* x, const void* w, const void* b, const void* residual, void* y,
                         int M, int N, int K, int act, int w_layout, void* stream);

/*
 * Weight-only int8 linear, the W-int8 / A-fp16 setting of the evaluation's largest model (Section 5.1):
 * symmetric per-output-channel quantisation, W(k,n) = scale[n] * w_int8[n,k]:
 *     y[m,n] = act(scale[n] * sum_k x[m,k] * w_int8[n,k] + b[n]) + residual[m,n]
 * x [M,K], b [N], residual [M,N], y [M,N] fp16; w_int8 [N,K] int8; scale [N] fp32; b and residual may be
 * NULL; act as in forge_linear_act.  The weights are widened to fp16 inside the kernel (exactly) and fed to
 * the tensor core; the scale is applied to the fp32 accumulator.  K must be a multiple of 16, N of 8.
 */
int forge_linear_act_w8a16(const void* x, const void* w_int8, const float* scale, const void* b,
                           const void* residual, void* y, int M, int N, int K, int act, void* stream);

/*
 * Gated MLP input of the 1B-8B decoder models of the evaluation (SwiGLU; Section 2, model overview): the
 * linear+silu pattern of the operator-fusion pass and the element-wise product with the second
 * projection, in one kernel:
 *     y[m,n] = silu(sum_k x[m,k] * Wg(k,n)) * (sum_k x[m,k] * Wu(k,n)),   silu(z) = z / (1 + exp(-z))
 * x [M,K], w_gate and w_up both [K,N] (FORGE_W_KN) or both [N,K] (FORGE_W_NK), y [M,N]; bf16 in and
 * out, fp32 accumulation; neither product reaches memory.  No bias (these models have none here).
 * K and N must be multiples of 8.  Errors as forge_linear_act.
 */
int forge_linear_swiglu(const void* x, const void* w_gate, const void* w_up, void* y,
                        int M, int N, int K, int w_layout, void* stream);

/*
 * Buffer planning for a fixed sequence of operators (Section 4.5, "Liveness Analysis" and "Linear-Scan
 * Buffer Allocation").  Host code only; nothing is launched.
 *
 * forge_plan_liveness (Eq. 14): the program is ops 0 .. num_ops-1; op j writes register out_reg[j] (-1: none)
 * and reads registers in_regs[in_off[j]] .. in_regs[in_off[j+1]-1].  On return start[r] is the op that
 * writes register r (-1 for a register nobody writes: an input) and end[r] the last op that reads it
 * (start[r] for a register that is never read).  FORGE_ERR_INVALID_ARG for a register index out of range
 * or a register with two writers.
 *
 * forge_plan_linear_scan (Algorithm 2): n live intervals [start[i], end[i]] (end >= start) are mapped to
 * buffers.  Intervals are taken in order of their start (ties by index); intervals that ended BEFORE the
 * current start (end < start) are expired and their buffers returned to a pool; the interval gets the
 * buffer released longest ago, or a new one if the pool is empty or pinned[i] is set (pinned may be NULL;
 * a pinned register's buffer goes to the pool like any other once the register has expired, as in the
 * paper's listing).  Two intervals that share an op index overlap and never share a buffer.  buf_of[i]
 * receives the buffer of interval i, *num_bufs the number M of buffers, buf_bytes[0..M-1] (if not NULL; room
 * for n entries) the size of each: the largest bytes[i] among its tenants (bytes may be NULL: all sizes 1).
 * The buffer reduction ratio of Eq. 15 is 1 - M / n.
 */
int forge_plan_liveness(int num_ops, const int* out_reg, const int* in_off, const int* in_regs,
                        int num_regs, int* start, int* end);
int forge_plan_linear_scan(int n, const int* start, const int* end, const size_t* bytes,
                           const unsigned char* pinned, int* buf_of, size_t* buf_bytes, int* num_bufs);

/*
 * A decoder layer run as a fixed sequence of the fused operators on one stream, with its intermediate
 * tensors in planned buffers (Section 4.5; the flat pre-resolved instruction stream of Listing 9):
 *     qkv  = x Wqkv (+ b_qkv)                                  [T, (Hq + 2 Hkv) D],  T = B S
 *     attn = fused attention over the q, k, v columns of qkv    [T, Hq D]   (mask_kind / lens / scale)
 *     h1   = attn Wo (+ b_o) + x                                [T, Hq D]
 *     g    = silu(h1 Wgate) * (h1 Wup)        (FORGE_MLP_SWIGLU; b_up must be NULL)
 *          | gelu_tanh(h1 Wup + b_up)         (FORGE_MLP_GELU; w_gate unused)          [T, F]
 *     y    = g Wdown (+ b_down) + h1                            [T, Hq D]
 * The columns of qkv are the Hq query heads, then the Hkv key heads, then the Hkv value heads, D each.
 * Normalisations and rotary embeddings, which the fusion passes leave alone, are not part of it.
 * x [T, Hq D] and y [T, Hq D] are the caller's bf16 device tensors; all weights bf16, every one stored
 * [in, out] (FORGE_W_KN) or every one [out, in] (FORGE_W_NK); biases [out] or NULL.  The four
 * intermediates live in `workspace` (256-byte aligned, at least forge_decoder_layer_workspace_bytes):
 * their live intervals let the linear scan put them into two buffers.  forge_decoder_layer_plan reports
 * the plan (N registers, M buffers, rho_buf = 1 - M/N, sizes and offsets) without launching anything.
 * D: a multiple of 8 up to 128; F a multiple of 8.  Errors as the operators'.
 */
enum { FORGE_MLP_SWIGLU = 0, FORGE_MLP_GELU = 1 };
typedef struct forge_decoder_layer_desc {
    int B, S, Hq, Hkv, D, F;
    int mlp_kind;   /* FORGE_MLP_SWIGLU or FORGE_MLP_GELU */
    int w_layout;   /* FORGE_W_KN or FORGE_W_NK, for every weight */
    int mask_kind;  /* FORGE_MASK_* for the attention */
    float scale;    /* of the attention scores */
    const int32_t* lens;  /* device, [B]; NULL unless mask_kind has the padding bit */
    const void *w_qkv, *b_qkv, *w_o, *b_o, *w_gate, *w_up, *b_up, *w_down, *b_down;
} forge_decoder_layer_desc;
typedef struct forge_layer_plan {
    int num_regs;          /* N: planned intermediates (qkv, attn, h1, g) */
    int num_bufs;          /* M */
    float rho_buf;         /* 1 - M / N (Eq. 15) */
    int buf_of[4];         /* buffer of each register */
    int reg_start[4], reg_end[4];   /* live intervals in op indices (Eq. 14) */
    size_t reg_bytes[4];
    size_t buf_bytes[4], buf_offset[4];  /* first num_bufs entries: size and place in the workspace */
    size_t workspace_bytes;  /* what the planned buffers take */
    size_t unplanned_bytes;  /* what one buffer per register would take */
} forge_layer_plan;
int forge_decoder_layer_plan(const forge_decoder_layer_desc* desc, forge_layer_plan* plan);
size_t forge_decoder_layer_workspace_bytes(const forge_decoder_layer_desc* desc);
int forge_decoder_layer(const forge_decoder_layer_desc* desc, const void* x, void* y,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * Host-buffer variants: the same operators for callers whose tensors live in
 * HOST memory (pinned memory makes the copies asynchronous).  Inputs are copied
 * to `dev_scratch`, the operator runs there, and the result is copied back to the
 * host pointer, all ordered after what `stream` held before the call and before
 * what it is given afterwards; the call returns without synchronising.  (The
 * 16-bit attention with several batch entries moves entry by entry on two streams
 * of the library's own, so that copies in, kernels and copies out overlap.)
 * dev_scratch is DEVICE memory of at least forge_*_host_scratch_bytes(...) bytes,
 * 256-byte aligned, owned by the caller.  `lens` is a HOST pointer here.
 */
size_t forge_attn_host_scratch_bytes(int B, int Hq, int Hkv, int Sq, int Skv, int D, int elem_bytes);
int forge_attn_fused_host(const void* q, const void* k, const void* v, void* out,
                          int B, int Hq, int Hkv, int Sq, int Skv, int D,
                          int mask_kind, const int32_t* lens, float scale,
                          void* dev_scratch, size_t dev_scratch_bytes, void* stream);
int forge_attn_fused_f32_host(const void* q, const void* k, const void* v, void* out,
                              int B, int Hq, int Hkv, int Sq, int Skv, int D,
                              int mask_kind, const int32_t* lens, float scale,
                              void* dev_scratch, size_t dev_scratch_bytes, void* stream);
size_t forge_attn_decode_host_scratch_bytes(int B, int Hq, int Hkv, int Smax, int D, int num_splits);
int forge_attn_decode_splitkv_host(const void* q, const void* k_cache, const void* v_cache, void* out,
                                   int B, int Hq, int Hkv, int Smax, int D,
                                   const int32_t* lens, int num_splits, float scale,
                                   void* dev_scratch, size_t dev_scratch_bytes, void* stream);
size_t forge_linear_host_scratch_bytes(int M, int N, int K);
int forge_linear_bias_gelu_host(const void* x, const void* w, const void* b, void* y,
                                int M, int N, int K,
                                void* dev_scratch, size_t dev_scratch_bytes, void* stream);

/*
 * Synchronises `stream`, then reports whether any kernel launched by this library
 * since the last call gave up on a bounded wait (FORGE_ERR_TIMEOUT) and clears the
 * flag.  Returns FORGE_OK otherwise, FORGE_ERR_CUDA if the stream itself failed.
 * The flag is one word per device, not per stream: a timeout raised by a kernel on
 * another stream of the same device is reported to (and cleared by) whichever caller
 * asks first, and only `stream` is synchronised.
 */
int forge_check_status(void* stream);

/*
 * The activation of the fused linear's epilogue (Eq. 11: the `act` of matmul -> bias add -> act),
 * applied element-wise: y[i] = act(x[i]) for i < n, fp32 device arrays (4-byte aligned), act one of
 * FORGE_ACT_*.  The kernels of forge_linear_* call the same device function on their fp32 accumulators,
 * so this entry point shows exactly which formula they use, at fp32 resolution (the 16-bit outputs of
 * the fused operators cannot separate tanh-GELU from erf-GELU).  exact = 0: as in the kernels
 * (exponential and reciprocal on the special-function unit); exact != 0: the same formulas with the
 * accurate library routines.  Errors: FORGE_ERR_INVALID_ARG, FORGE_ERR_CUDA.
 */
int forge_activation_f32(const float* x, float* y, size_t n, int act, int exact, void* stream);

/*
 * Exercises the failure path of the bounded waits (every wait inside the kernels gives up after a
 * clock budget, sets the device's status word and lets the kernel return): launches one warp that
 * waits, with the kernels' own wait routine and a budget of `budget_clocks` SM clocks
 * (0 .. 200,000,000), for a barrier nothing ever completes.  After the budget the warp sets the
 * status word and exits; the next forge_check_status() returns FORGE_ERR_TIMEOUT and the one after
 * that FORGE_OK.  Nothing else is touched; no operator kernel is involved.  The paper has no
 * counterpart: this is a self-test of the library's error reporting.
 */
int forge_debug_wait_timeout(long long budget_clocks, void* stream);

/* Human-readable name of a forge_status value (static storage). */
const char* forge_status_string(int status);

/* The cudaError_t (as int) behind the most recent FORGE_ERR_CUDA on this thread. */
int forge_last_cuda_error(void);

/* Number of kernels this library has launched in this process (for accounting). */
unsigned long long forge_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FORGE_H_ */
