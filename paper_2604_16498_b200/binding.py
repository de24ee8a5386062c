"""Python binding of the C ABI in ``include/forge.h`` (argument marshalling only).

Every function takes torch tensors (used purely as owners of device or pinned host
memory), checks shapes and dtypes, and passes raw pointers, sizes and the current
CUDA stream to ``libforge.so``.  All arithmetic happens inside the library's kernels.
There is no fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libforge.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
MASK_NONE, MASK_CAUSAL, MASK_PADDING, MASK_CAUSAL_PADDING = range(4)

# name -> (restype, argtypes); mirrors include/forge.h
_vp, _i, _f, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
_ATTN = [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i, _vp, _f]
_DEC = [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _i, _f]
SIGNATURES = {
    "forge_attn_fused": (_i, _ATTN + [_vp]),
    "forge_attn_fused_f32": (_i, _ATTN + [_vp]),
    "forge_attn_fused_f16": (_i, _ATTN + [_vp]),
    "forge_attn_fused_strided": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _i, _vp, _f, _vp]),
    "forge_attn_fused_bias": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i, _vp, _vp, _i, _f, _vp]),
    "forge_attn_decode_splitkv": (_i, _DEC + [_vp, _sz, _vp]),
    "forge_attn_decode_splitkv_f16": (_i, _DEC + [_vp, _sz, _vp]),
    "forge_attn_decode_workspace_bytes": (_sz, [_i, _i, _i, _i]),
    "forge_attn_decode_workspace_init": (_i, [_vp, _sz, _vp]),
    "forge_attn_decode_splitkv_static": (_i, _DEC + [_vp]),
    "forge_linear_bias_gelu": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "forge_linear_act": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]),
    "forge_linear_act_f16": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]),
    "forge_linear_act_w8a16": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp]),
    "forge_linear_swiglu": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp]),
    "forge_attn_host_scratch_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _i]),
    "forge_attn_fused_host": (_i, _ATTN + [_vp, _sz, _vp]),
    "forge_attn_fused_f32_host": (_i, _ATTN + [_vp, _sz, _vp]),
    "forge_attn_decode_host_scratch_bytes": (_sz, [_i, _i, _i, _i, _i, _i]),
    "forge_attn_decode_splitkv_host": (_i, _DEC + [_vp, _sz, _vp]),
    "forge_linear_host_scratch_bytes": (_sz, [_i, _i, _i]),
    "forge_linear_bias_gelu_host": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "forge_check_status": (_i, [_vp]),
    "forge_activation_f32": (_i, [_vp, _vp, _sz, _i, _i, _vp]),
    "forge_debug_wait_timeout": (_i, [ctypes.c_longlong, _vp]),
    "forge_status_string": (ctypes.c_char_p, [_i]),
    "forge_last_cuda_error": (_i, []),
    "forge_launch_count": (ctypes.c_ulonglong, []),
}



class LayerDesc(ctypes.Structure):
    """forge_decoder_layer_desc"""
    _fields_ = [("B", _i), ("S", _i), ("Hq", _i), ("Hkv", _i), ("D", _i), ("F", _i), ("mlp_kind", _i),
                ("w_layout", _i), ("mask_kind", _i), ("scale", _f), ("lens", _vp),
                ("w_qkv", _vp), ("b_qkv", _vp), ("w_o", _vp), ("b_o", _vp), ("w_gate", _vp), ("w_up", _vp),
                ("b_up", _vp), ("w_down", _vp), ("b_down", _vp)]


class LayerPlan(ctypes.Structure):
    """forge_layer_plan"""
    _fields_ = [("num_regs", _i), ("num_bufs", _i), ("rho_buf", _f), ("buf_of", _i * 4), ("reg_start", _i * 4),
                ("reg_end", _i * 4), ("reg_bytes", _sz * 4), ("buf_bytes", _sz * 4), ("buf_offset", _sz * 4),
                ("workspace_bytes", _sz), ("unplanned_bytes", _sz)]


SIGNATURES.update({
    "forge_plan_liveness": (_i, [_i, _vp, _vp, _vp, _i, _vp, _vp]),
    "forge_plan_linear_scan": (_i, [_i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "forge_decoder_layer_plan": (_i, [ctypes.POINTER(LayerDesc), ctypes.POINTER(LayerPlan)]),
    "forge_decoder_layer_workspace_bytes": (_sz, [ctypes.POINTER(LayerDesc)]),
    "forge_decoder_layer": (_i, [ctypes.POINTER(LayerDesc), _vp, _vp, _vp, _sz, _vp]),
})

_lib = None


class ForgeError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        lib = load()
        name = lib.forge_status_string(status).decode()
        extra = f" (cudaError {lib.forge_last_cuda_error()})" if status == ERR_CUDA else ""
        super().__init__(f"{fn} failed: {name}{extra}")


def load() -> ctypes.CDLL:
    """Loads ``libforge.so`` (built by ``paper_2604_16498_b200.build``).  Raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_16498_b200.build` "
                               "(there is no fallback implementation)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _host(t: torch.Tensor, dtype, name: str) -> int:
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name}: expected a contiguous host tensor of {dtype}")
    return t.data_ptr()


def _check(fn: str, status: int) -> None:
    if status != OK:
        raise ForgeError(fn, status)


def _attn_dims(q, k, v):
    B, Hq, Sq, D = q.shape
    Bk, Hkv, Skv, Dk = k.shape
    if (Bk, Dk) != (B, D) or tuple(v.shape) != tuple(k.shape):
        raise ValueError("q [B,Hq,Sq,D], k/v [B,Hkv,Skv,D] expected")
    return B, Hq, Hkv, Sq, Skv, D


def attn_fused(q, k, v, mask_kind=MASK_NONE, lens=None, scale=None, out=None):
    """forge_attn_fused: bf16 tensors q [B,Hq,Sq,D], k/v [B,Hkv,Skv,D] on the GPU."""
    B, Hq, Hkv, Sq, Skv, D = _attn_dims(q, k, v)
    out = torch.empty_like(q) if out is None else out
    scale = D ** -0.5 if scale is None else scale
    lp = None if lens is None else _dev(lens, torch.int32, "lens")
    _check("forge_attn_fused", load().forge_attn_fused(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(out, torch.bfloat16, "out"), B, Hq, Hkv, Sq, Skv, D, int(mask_kind), lp, float(scale), _stream()))
    return out


def attn_fused_strided(q, k, v, out, mask_kind=MASK_NONE, lens=None, scale=None):
    """forge_attn_fused_strided: q/out [B,Hq,Sq,D] and k/v [B,Hkv,Skv,D] bf16 VIEWS (any strides with a
    contiguous last dimension, e.g. slices of a fused QKV projection permuted to head-major)."""
    B, Hq, Sq, D = q.shape
    _, Hkv, Skv, _ = k.shape
    if tuple(k.shape) != (B, Hkv, Skv, D) or tuple(v.shape) != (B, Hkv, Skv, D) or tuple(out.shape) != (B, Hq, Sq, D):
        raise ValueError("q/out [B,Hq,Sq,D], k/v [B,Hkv,Skv,D] expected")
    scale = D ** -0.5 if scale is None else scale
    arrs = []
    for name, t in (("q", q), ("k", k), ("v", v), ("out", out)):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.stride(3) == 1):
            raise ValueError(f"{name}: expected a CUDA bf16 tensor whose last dimension is contiguous")
        arrs.append((ctypes.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2)))
    lp = None if lens is None else _dev(lens, torch.int32, "lens")
    _check("forge_attn_fused_strided", load().forge_attn_fused_strided(
        q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), B, Hq, Hkv, Sq, Skv, D,
        arrs[0], arrs[1], arrs[2], arrs[3], int(mask_kind), lp, float(scale), _stream()))
    return out


def attn_fused_f16(q, k, v, mask_kind=MASK_NONE, lens=None, scale=None, out=None):
    """forge_attn_fused_f16: the same operator on fp16 tensors."""
    B, Hq, Hkv, Sq, Skv, D = _attn_dims(q, k, v)
    out = torch.empty_like(q) if out is None else out
    scale = D ** -0.5 if scale is None else scale
    lp = None if lens is None else _dev(lens, torch.int32, "lens")
    _check("forge_attn_fused_f16", load().forge_attn_fused_f16(
        _dev(q, torch.float16, "q"), _dev(k, torch.float16, "k"), _dev(v, torch.float16, "v"),
        _dev(out, torch.float16, "out"), B, Hq, Hkv, Sq, Skv, D, int(mask_kind), lp, float(scale), _stream()))
    return out


def attn_fused_bias(q, k, v, bias, mask_kind=MASK_NONE, lens=None, scale=None, out=None):
    """forge_attn_fused_bias: bf16 q/k/v and an fp32 additive bias [B, 1 or Hq, Sq, Skv] on the scaled scores."""
    B, Hq, Hkv, Sq, Skv, D = _attn_dims(q, k, v)
    if bias.dim() != 4 or bias.shape[0] != B or bias.shape[2] != Sq or bias.shape[3] != Skv:
        raise ValueError("bias [B, 1 or Hq, Sq, Skv] expected")
    out = torch.empty_like(q) if out is None else out
    scale = D ** -0.5 if scale is None else scale
    lp = None if lens is None else _dev(lens, torch.int32, "lens")
    _check("forge_attn_fused_bias", load().forge_attn_fused_bias(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(out, torch.bfloat16, "out"), B, Hq, Hkv, Sq, Skv, D, int(mask_kind), lp,
        _dev(bias, torch.float32, "bias"), int(bias.shape[1]), float(scale), _stream()))
    return out


def attn_fused_f32(q, k, v, mask_kind=MASK_NONE, lens=None, scale=None, out=None):
    """forge_attn_fused_f32: the same operator on fp32 tensors."""
    B, Hq, Hkv, Sq, Skv, D = _attn_dims(q, k, v)
    out = torch.empty_like(q) if out is None else out
    scale = D ** -0.5 if scale is None else scale
    lp = None if lens is None else _dev(lens, torch.int32, "lens")
    _check("forge_attn_fused_f32", load().forge_attn_fused_f32(
        _dev(q, torch.float32, "q"), _dev(k, torch.float32, "k"), _dev(v, torch.float32, "v"),
        _dev(out, torch.float32, "out"), B, Hq, Hkv, Sq, Skv, D, int(mask_kind), lp, float(scale), _stream()))
    return out


def attn_decode_workspace_bytes(B, Hq, D, num_splits) -> int:
    return int(load().forge_attn_decode_workspace_bytes(B, Hq, D, num_splits))


def attn_decode_workspace_init(workspace) -> None:
    """forge_attn_decode_workspace_init: clears a new decode workspace (its arrival counters must start at zero)."""
    _check("forge_attn_decode_workspace_init", load().forge_attn_decode_workspace_init(
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()))


def attn_decode_splitkv(q, k_cache, v_cache, lens, num_splits, scale=None, out=None, workspace=None):
    """forge_attn_decode_splitkv (bf16 tensors) or forge_attn_decode_splitkv_f16 (fp16 tensors), chosen by
    q.dtype: q [B,Hq,D], caches [B,Hkv,Smax,D], lens int32 [B].  A workspace passed in must have been
    cleared once (attn_decode_workspace_init); without one, a fresh cleared workspace is allocated."""
    B, Hq, D = q.shape
    Bk, Hkv, Smax, Dk = k_cache.shape
    if (Bk, Dk) != (B, D) or tuple(v_cache.shape) != tuple(k_cache.shape):
        raise ValueError("q [B,Hq,D], caches [B,Hkv,Smax,D] expected")
    out = torch.empty_like(q) if out is None else out
    scale = D ** -0.5 if scale is None else scale
    need = attn_decode_workspace_bytes(B, Hq, D, num_splits)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
        attn_decode_workspace_init(workspace)
    dt = torch.float16 if q.dtype == torch.float16 else torch.bfloat16
    name = "forge_attn_decode_splitkv_f16" if dt == torch.float16 else "forge_attn_decode_splitkv"
    _check(name, getattr(load(), name)(
        _dev(q, dt, "q"), _dev(k_cache, dt, "k_cache"),
        _dev(v_cache, dt, "v_cache"), _dev(out, dt, "out"),
        B, Hq, Hkv, Smax, D, _dev(lens, torch.int32, "lens"), int(num_splits), float(scale),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()))
    return out


DECODE_STATIC_SCRATCH_BYTES = 8 << 20


def attn_decode_splitkv_static(q, k_cache, v_cache, lens, num_splits, out, scale=None):
    """forge_attn_decode_splitkv_static: the decode step for callers that cannot allocate a
    workspace.  The partials go to a fixed 8 MiB array inside the library (shared by all calls on
    the device, so calls must not overlap); larger problems raise ForgeError(ERR_WORKSPACE).
    `out` is the caller's buffer: nothing is allocated here either."""
    B, Hq, D = q.shape
    Bk, Hkv, Smax, Dk = k_cache.shape
    if (Bk, Dk) != (B, D) or tuple(v_cache.shape) != tuple(k_cache.shape):
        raise ValueError("q [B,Hq,D], caches [B,Hkv,Smax,D] expected")
    scale = D ** -0.5 if scale is None else scale
    _check("forge_attn_decode_splitkv_static", load().forge_attn_decode_splitkv_static(
        _dev(q, torch.bfloat16, "q"), _dev(k_cache, torch.bfloat16, "k_cache"),
        _dev(v_cache, torch.bfloat16, "v_cache"), _dev(out, torch.bfloat16, "out"),
        B, Hq, Hkv, Smax, D, _dev(lens, torch.int32, "lens"), int(num_splits), float(scale), _stream()))
    return out


def linear_bias_gelu(x, w, b, out=None):
    """forge_linear_bias_gelu: x [M,K], w [K,N], b [N] (bf16) -> gelu_tanh(x @ w + b) [M,N]."""
    M, K = x.shape
    K2, N = w.shape
    if K2 != K or tuple(b.shape) != (N,):
        raise ValueError("x [M,K], w [K,N], b [N] expected")
    out = torch.empty((M, N), dtype=torch.bfloat16, device=x.device) if out is None else out
    _check("forge_linear_bias_gelu", load().forge_linear_bias_gelu(
        _dev(x, torch.bfloat16, "x"), _dev(w, torch.bfloat16, "w"), _dev(b, torch.bfloat16, "b"),
        _dev(out, torch.bfloat16, "out"), M, N, K, _stream()))
    return out


ACT_GELU_TANH, ACT_GELU_ERF, ACT_RELU, ACT_SILU, ACT_NONE = range(5)
W_KN, W_NK = 0, 1


def linear_act(x, w, b=None, residual=None, act=ACT_GELU_TANH, w_layout=W_KN, out=None):
    """forge_linear_act (bf16 tensors) or forge_linear_act_f16 (fp16 tensors), chosen by x.dtype:
    act(x @ W + b) + residual with W given as [K,N] (W_KN) or [N,K] (W_NK)."""
    M, K = x.shape
    N = w.shape[1] if w_layout == W_KN else w.shape[0]
    if tuple(w.shape) != ((K, N) if w_layout == W_KN else (N, K)):
        raise ValueError("w must be [K,N] for W_KN and [N,K] for W_NK")
    if b is not None and tuple(b.shape) != (N,):
        raise ValueError("b [N] expected")
    if residual is not None and tuple(residual.shape) != (M, N):
        raise ValueError("residual [M,N] expected")
    out = torch.empty((M, N), dtype=x.dtype, device=x.device) if out is None else out
    bf = torch.float16 if x.dtype == torch.float16 else torch.bfloat16
    name = "forge_linear_act_f16" if bf == torch.float16 else "forge_linear_act"
    _check(name, getattr(load(), name)(
        _dev(x, bf, "x"), _dev(w, bf, "w"), None if b is None else _dev(b, bf, "b"),
        None if residual is None else _dev(residual, bf, "residual"), _dev(out, bf, "out"),
        M, N, K, int(act), int(w_layout), _stream()))
    return out


def linear_act_w8a16(x, w_int8, scale, b=None, residual=None, act=ACT_GELU_TANH, out=None):
    """forge_linear_act_w8a16: fp16 x [M,K], int8 weights [N,K], fp32 per-channel scale [N]."""
    M, K = x.shape
    N = w_int8.shape[0]
    if tuple(w_int8.shape) != (N, K) or tuple(scale.shape) != (N,):
        raise ValueError("w_int8 [N,K] and scale [N] expected")
    out = torch.empty((M, N), dtype=torch.float16, device=x.device) if out is None else out
    h = torch.float16
    _check("forge_linear_act_w8a16", load().forge_linear_act_w8a16(
        _dev(x, h, "x"), _dev(w_int8, torch.int8, "w_int8"), _dev(scale, torch.float32, "scale"),
        None if b is None else _dev(b, h, "b"), None if residual is None else _dev(residual, h, "residual"),
        _dev(out, h, "out"), M, N, K, int(act), _stream()))
    return out


def linear_swiglu(x, w_gate, w_up, w_layout=W_KN, out=None):
    """forge_linear_swiglu: silu(x @ Wg) * (x @ Wu); both weights [K,N] (W_KN) or [N,K] (W_NK)."""
    M, K = x.shape
    N = w_gate.shape[1] if w_layout == W_KN else w_gate.shape[0]
    want = (K, N) if w_layout == W_KN else (N, K)
    if tuple(w_gate.shape) != want or tuple(w_up.shape) != want:
        raise ValueError("w_gate and w_up must both be [K,N] for W_KN or [N,K] for W_NK")
    out = torch.empty((M, N), dtype=torch.bfloat16, device=x.device) if out is None else out
    bf = torch.bfloat16
    _check("forge_linear_swiglu", load().forge_linear_swiglu(
        _dev(x, bf, "x"), _dev(w_gate, bf, "w_gate"), _dev(w_up, bf, "w_up"), _dev(out, bf, "out"),
        M, N, K, int(w_layout), _stream()))
    return out


# ---- buffer planning (host only) and the decoder layer ----
MLP_SWIGLU, MLP_GELU = 0, 1


def plan_liveness(out_reg, in_regs_per_op, num_regs):
    """forge_plan_liveness: ops given as (register written or -1, list of registers read).  Returns (start, end)."""
    n = len(out_reg)
    off = [0]
    flat = []
    for regs in in_regs_per_op:
        flat.extend(regs)
        off.append(len(flat))
    c_out = (ctypes.c_int * max(n, 1))(*out_reg)
    c_off = (ctypes.c_int * (n + 1))(*off)
    c_in = (ctypes.c_int * max(len(flat), 1))(*flat)
    start = (ctypes.c_int * max(num_regs, 1))()
    end = (ctypes.c_int * max(num_regs, 1))()
    _check("forge_plan_liveness", load().forge_plan_liveness(n, c_out, c_off, c_in, num_regs, start, end))
    return list(start)[:num_regs], list(end)[:num_regs]


def plan_linear_scan(start, end, nbytes=None, pinned=None):
    """forge_plan_linear_scan.  Returns (buf_of, buf_bytes, num_bufs)."""
    n = len(start)
    c_s = (ctypes.c_int * max(n, 1))(*start)
    c_e = (ctypes.c_int * max(n, 1))(*end)
    c_b = None if nbytes is None else (ctypes.c_size_t * max(n, 1))(*nbytes)
    c_p = None if pinned is None else (ctypes.c_ubyte * max(n, 1))(*[1 if x else 0 for x in pinned])
    buf_of = (ctypes.c_int * max(n, 1))()
    buf_bytes = (ctypes.c_size_t * max(n, 1))()
    m = ctypes.c_int(0)
    _check("forge_plan_linear_scan", load().forge_plan_linear_scan(n, c_s, c_e, c_b, c_p, buf_of, buf_bytes, ctypes.byref(m)))
    return list(buf_of)[:n], list(buf_bytes)[:m.value], m.value


def _layer_desc(B, S, Hq, Hkv, D, F, mlp_kind, w_layout, mask_kind, scale, lens, weights):
    d = LayerDesc(B=B, S=S, Hq=Hq, Hkv=Hkv, D=D, F=F, mlp_kind=mlp_kind, w_layout=w_layout, mask_kind=mask_kind,
                  scale=float(scale), lens=None if lens is None else _dev(lens, torch.int32, "lens"))
    for name in ("w_qkv", "b_qkv", "w_o", "b_o", "w_gate", "w_up", "b_up", "w_down", "b_down"):
        t = weights.get(name)
        setattr(d, name, None if t is None else _dev(t, torch.bfloat16, name))
    return d


def decoder_layer_plan(B, S, Hq, Hkv, D, F, mlp_kind=MLP_SWIGLU):
    """forge_decoder_layer_plan: the buffer plan of a layer of these dimensions (no GPU needed)."""
    d = LayerDesc(B=B, S=S, Hq=Hq, Hkv=Hkv, D=D, F=F, mlp_kind=mlp_kind, w_layout=W_KN, mask_kind=MASK_CAUSAL, scale=1.0)
    plan = LayerPlan()
    _check("forge_decoder_layer_plan", load().forge_decoder_layer_plan(ctypes.byref(d), ctypes.byref(plan)))
    return plan


def decoder_layer(x, weights, B, S, Hq, Hkv, D, F, mlp_kind=MLP_SWIGLU, w_layout=W_KN, mask_kind=MASK_CAUSAL,
                  scale=None, lens=None, out=None, workspace=None):
    """forge_decoder_layer: x [B*S, Hq*D] bf16; weights: dict of bf16 tensors (w_qkv, w_o, w_gate, w_up, w_down
    and optional b_qkv, b_o, b_up, b_down)."""
    scale = D ** -0.5 if scale is None else scale
    d = _layer_desc(B, S, Hq, Hkv, D, F, mlp_kind, w_layout, mask_kind, scale, lens, weights)
    out = torch.empty_like(x) if out is None else out
    need = int(load().forge_decoder_layer_workspace_bytes(ctypes.byref(d)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    _check("forge_decoder_layer", load().forge_decoder_layer(
        ctypes.byref(d), _dev(x, torch.bfloat16, "x"), _dev(out, torch.bfloat16, "out"),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()))
    return out


# ---- host-buffer variants: tensors in (pinned) host memory, device scratch from the caller ----
def attn_host_scratch_bytes(B, Hq, Hkv, Sq, Skv, D, elem_bytes) -> int:
    return int(load().forge_attn_host_scratch_bytes(B, Hq, Hkv, Sq, Skv, D, elem_bytes))


def attn_fused_host(q, k, v, out, scratch, mask_kind=MASK_NONE, lens=None, scale=None):
    """forge_attn_fused_host / forge_attn_fused_f32_host, chosen by q.dtype.  Asynchronous."""
    B, Hq, Hkv, Sq, Skv, D = _attn_dims(q, k, v)
    f32 = q.dtype == torch.float32
    dt = torch.float32 if f32 else torch.bfloat16
    scale = D ** -0.5 if scale is None else scale
    lp = None if lens is None else _host(lens, torch.int32, "lens")
    fn = "forge_attn_fused_f32_host" if f32 else "forge_attn_fused_host"
    _check(fn, getattr(load(), fn)(
        _host(q, dt, "q"), _host(k, dt, "k"), _host(v, dt, "v"), _host(out, dt, "out"),
        B, Hq, Hkv, Sq, Skv, D, int(mask_kind), lp, float(scale),
        _dev(scratch, torch.uint8, "scratch"), scratch.numel(), _stream()))
    return out


def attn_decode_host_scratch_bytes(B, Hq, Hkv, Smax, D, num_splits) -> int:
    return int(load().forge_attn_decode_host_scratch_bytes(B, Hq, Hkv, Smax, D, num_splits))


def attn_decode_splitkv_host(q, k_cache, v_cache, lens, num_splits, out, scratch, scale=None):
    B, Hq, D = q.shape
    _, Hkv, Smax, _ = k_cache.shape
    scale = D ** -0.5 if scale is None else scale
    bf = torch.bfloat16
    _check("forge_attn_decode_splitkv_host", load().forge_attn_decode_splitkv_host(
        _host(q, bf, "q"), _host(k_cache, bf, "k_cache"), _host(v_cache, bf, "v_cache"), _host(out, bf, "out"),
        B, Hq, Hkv, Smax, D, _host(lens, torch.int32, "lens"), int(num_splits), float(scale),
        _dev(scratch, torch.uint8, "scratch"), scratch.numel(), _stream()))
    return out


def linear_host_scratch_bytes(M, N, K) -> int:
    return int(load().forge_linear_host_scratch_bytes(M, N, K))


def linear_bias_gelu_host(x, w, b, out, scratch):
    M, K = x.shape
    _, N = w.shape
    bf = torch.bfloat16
    _check("forge_linear_bias_gelu_host", load().forge_linear_bias_gelu_host(
        _host(x, bf, "x"), _host(w, bf, "w"), _host(b, bf, "b"), _host(out, bf, "out"), M, N, K,
        _dev(scratch, torch.uint8, "scratch"), scratch.numel(), _stream()))
    return out


def activation_f32(x, act, exact=False, out=None):
    """forge_activation_f32: the fused linear's epilogue activation, element-wise on an fp32 CUDA tensor."""
    out = torch.empty_like(x) if out is None else out
    _check("forge_activation_f32", load().forge_activation_f32(
        _dev(x, torch.float32, "x"), _dev(out, torch.float32, "out"), x.numel(), int(act), int(bool(exact)), _stream()))
    return out


def debug_wait_timeout(budget_clocks: int = 1_000_000) -> None:
    """forge_debug_wait_timeout: one warp runs the kernels' bounded wait on a barrier nothing completes."""
    _check("forge_debug_wait_timeout", load().forge_debug_wait_timeout(int(budget_clocks), _stream()))


def check_status() -> None:
    """Synchronises the current stream and raises if a kernel gave up on a bounded wait."""
    _check("forge_check_status", load().forge_check_status(_stream()))


def launch_count() -> int:
    return int(load().forge_launch_count())
