// A whole decoder layer from the fused operators, run as a fixed sequence on one stream into planned
// buffers (Section 4.5: liveness, linear-scan buffer allocation, and the flat pre-resolved instruction
// stream of the compiled executor, Listing 9).  The layer is what the attention-fusion and
// operator-fusion passes leave of a transformer block (normalisations and rotary embeddings, which
// those passes do not touch, are not part of it):
//
//   op 0   qkv  = x Wqkv (+ b)                       fused linear            [T, (Hq + 2 Hkv) D]
//   op 1   attn = softmax(scale q k^T + mask) v      fused attention, reading q, k, v as strided views of
//                                                    qkv and writing token-major rows      [T, Hq D]
//   op 2   h1   = attn Wo (+ b) + x                  mm+add                  [T, Hq D]
//   op 3   g    = silu(h1 Wg) * (h1 Wu)              gated MLP input         [T, F]
//            or   gelu_tanh(h1 W1 + b1)              GPT-2 style
//   op 4   y    = g Wd (+ b) + h1                    mm+add                  [T, Hq D]
//
// x and y belong to the caller; qkv, attn, h1 and g are the registers that get planned: their live
// intervals are [0,1], [1,2], [2,4], [3,4], so the linear scan maps the four of them to two buffers.
// All launches are chained with programmatic stream serialisation by the operators themselves; nothing
// is allocated, looked up or decided at run time beyond this fixed list.
#include <algorithm>

#include "forge_common.cuh"

namespace forge {
namespace {

constexpr int kRegs = 4;  // qkv, attn, h1, g
inline size_t up256(size_t n) { return (n + 255) & ~(size_t)255; }

int check_desc(const forge_decoder_layer_desc* d) {
    if (!d) return FORGE_ERR_INVALID_ARG;
    if (d->B <= 0 || d->S <= 0 || d->Hq <= 0 || d->Hkv <= 0 || d->D <= 0 || d->F <= 0) return FORGE_ERR_INVALID_ARG;
    if (d->Hq % d->Hkv != 0) return FORGE_ERR_INVALID_ARG;
    if (d->mlp_kind != FORGE_MLP_SWIGLU && d->mlp_kind != FORGE_MLP_GELU) return FORGE_ERR_INVALID_ARG;
    if (d->w_layout != FORGE_W_KN && d->w_layout != FORGE_W_NK) return FORGE_ERR_INVALID_ARG;
    if (d->mask_kind < 0 || d->mask_kind > 3) return FORGE_ERR_INVALID_ARG;
    if ((d->D % 8) != 0 || d->D > 128 || (d->F % 8) != 0) return FORGE_ERR_UNSUPPORTED;
    if ((long long)d->B * d->S > 2147483647LL) return FORGE_ERR_UNSUPPORTED;
    return FORGE_OK;
}

// Sizes of the four registers, their plan and their places in the workspace.
int make_plan(const forge_decoder_layer_desc* d, forge_layer_plan* plan) {
    const size_t T = (size_t)d->B * d->S, H = (size_t)d->Hq * d->D;
    const size_t bytes[kRegs] = {T * (size_t)(d->Hq + 2 * d->Hkv) * d->D * 2, T * H * 2, T * H * 2, T * (size_t)d->F * 2};
    // the instruction list in terms of registers: 0 = x (the caller's), 1..4 = qkv, attn, h1, g, 5 = y (the caller's)
    const int out_reg[5] = {1, 2, 3, 4, 5};
    const int in_off[6] = {0, 1, 2, 4, 5, 7};
    const int in_regs[7] = {0, 1, 2, 0, 3, 4, 3};
    int start[6], end[6];
    int st = forge_plan_liveness(5, out_reg, in_off, in_regs, 6, start, end);
    if (st != FORGE_OK) return st;
    size_t buf_bytes[kRegs];
    st = forge_plan_linear_scan(kRegs, start + 1, end + 1, bytes, nullptr, plan->buf_of, buf_bytes, &plan->num_bufs);
    if (st != FORGE_OK) return st;
    plan->num_regs = kRegs;
    plan->rho_buf = 1.0f - (float)plan->num_bufs / (float)kRegs;  // Eq. 15
    size_t off = 0, unplanned = 0;
    for (int b = 0; b < kRegs; ++b) {
        plan->buf_bytes[b] = b < plan->num_bufs ? buf_bytes[b] : 0;
        plan->buf_offset[b] = off;
        if (b < plan->num_bufs) off += up256(buf_bytes[b]);
    }
    for (int r = 0; r < kRegs; ++r) {
        plan->reg_bytes[r] = bytes[r];
        plan->reg_start[r] = start[r + 1];
        plan->reg_end[r] = end[r + 1];
        unplanned += up256(bytes[r]);
    }
    plan->workspace_bytes = off;
    plan->unplanned_bytes = unplanned;
    return FORGE_OK;
}

}  // namespace
}  // namespace forge

extern "C" int forge_decoder_layer_plan(const forge_decoder_layer_desc* desc, forge_layer_plan* plan) {
    using namespace forge;
    if (!plan) return FORGE_ERR_INVALID_ARG;
    const int st = check_desc(desc);
    if (st != FORGE_OK) return st;
    return make_plan(desc, plan);
}

extern "C" size_t forge_decoder_layer_workspace_bytes(const forge_decoder_layer_desc* desc) {
    forge_layer_plan plan;
    if (forge_decoder_layer_plan(desc, &plan) != FORGE_OK) return 0;
    return plan.workspace_bytes;
}

extern "C" int forge_decoder_layer(const forge_decoder_layer_desc* d, const void* x, void* y, void* workspace,
                                   size_t workspace_bytes, void* stream) {
    using namespace forge;
    int st = check_desc(d);
    if (st != FORGE_OK) return st;
    if (!x || !y || !workspace || !d->w_qkv || !d->w_o || !d->w_up || !d->w_down) return FORGE_ERR_INVALID_ARG;
    if (d->mlp_kind == FORGE_MLP_SWIGLU && (!d->w_gate || d->b_up)) return FORGE_ERR_INVALID_ARG;
    if ((d->mask_kind & FORGE_MASK_PADDING) && !d->lens) return FORGE_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return FORGE_ERR_INVALID_ARG;
    forge_layer_plan plan;
    st = make_plan(d, &plan);
    if (st != FORGE_OK) return st;
    if (workspace_bytes < plan.workspace_bytes) return FORGE_ERR_WORKSPACE;

    char* ws = static_cast<char*>(workspace);
    auto reg = [&](int r) { return static_cast<void*>(ws + plan.buf_offset[plan.buf_of[r]]); };
    uint16_t* qkv = static_cast<uint16_t*>(reg(0));
    void* attn = reg(1);
    void* h1 = reg(2);
    void* g = reg(3);
    const int T = d->B * d->S, H = d->Hq * d->D, Nqkv = (d->Hq + 2 * d->Hkv) * d->D;

    // op 0: fused QKV projection
    st = forge_linear_act(x, d->w_qkv, d->b_qkv, nullptr, qkv, T, Nqkv, H, FORGE_ACT_NONE, d->w_layout, stream);
    if (st != FORGE_OK) return st;
    // op 1: attention on views of qkv ([B, S, heads, D] seen as [B, heads, S, D]); token-major output
    const int64_t s_qkv[3] = {(int64_t)d->S * Nqkv, d->D, Nqkv};
    const int64_t s_out[3] = {(int64_t)d->S * H, d->D, H};
    st = forge_attn_fused_strided(qkv, qkv + (size_t)d->Hq * d->D, qkv + (size_t)(d->Hq + d->Hkv) * d->D, attn, d->B,
                                  d->Hq, d->Hkv, d->S, d->S, d->D, s_qkv, s_qkv, s_qkv, s_out, d->mask_kind, d->lens,
                                  d->scale, stream);
    if (st != FORGE_OK) return st;
    // op 2: output projection + residual
    st = forge_linear_act(attn, d->w_o, d->b_o, x, h1, T, H, H, FORGE_ACT_NONE, d->w_layout, stream);
    if (st != FORGE_OK) return st;
    // op 3: MLP input
    if (d->mlp_kind == FORGE_MLP_SWIGLU)
        st = forge_linear_swiglu(h1, d->w_gate, d->w_up, g, T, d->F, H, d->w_layout, stream);
    else
        st = forge_linear_act(h1, d->w_up, d->b_up, nullptr, g, T, d->F, H, FORGE_ACT_GELU_TANH, d->w_layout, stream);
    if (st != FORGE_OK) return st;
    // op 4: down projection + residual
    return forge_linear_act(g, d->w_down, d->b_down, h1, y, T, H, d->F, FORGE_ACT_NONE, d->w_layout, stream);
}
