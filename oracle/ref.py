"""ctypes binding for ``forge_ref.c`` (the CPU oracle).  Test infrastructure only.

Arrays are numpy fp64, C-contiguous; ``lens`` is int32.  Shapes follow the C file:
q/out [B,Hq,Sq,D], k/v [B,Hkv,Skv,D]; decode q/out [B,Hq,D], caches [B,Hkv,Smax,D];
linear x [M,K], w [K,N], b [N].
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "forge_ref.c")
_LIB = os.path.join(_HERE, "libforge_ref.so")
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math) if it is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _configure(lib):
    i = ctypes.c_int
    lib.forge_ref_attn.argtypes = [_dp, _dp, _dp, _dp, i, i, i, i, i, i, i, _ip, ctypes.c_double]
    lib.forge_ref_attn_probs.argtypes = [_dp, _dp, _dp, _dp, _dp, i, i, i, i, i, i, i, _ip, ctypes.c_double]
    lib.forge_ref_attn_bias.argtypes = [_dp, _dp, _dp, _dp, _dp, i, i, i, i, i, i, i, _ip, ctypes.c_double, _dp, i]
    lib.forge_ref_attn_decode.argtypes = [_dp, _dp, _dp, _dp, i, i, i, i, i, _ip, ctypes.c_double]
    lib.forge_ref_linear_bias_gelu.argtypes = [_dp, _dp, _dp, _dp, i, i, i]
    lib.forge_ref_linear_act.argtypes = [_dp, _dp, _dp, _dp, _dp, i, i, i, i, i]
    lib.forge_ref_linear_w8.argtypes = [_dp, _dp, _dp, _dp, _dp, _dp, i, i, i, i]
    lib.forge_ref_linear_swiglu.argtypes = [_dp, _dp, _dp, _dp, i, i, i, i]
    lib.forge_ref_gelu_tanh.argtypes = [ctypes.c_double]
    lib.forge_ref_gelu_tanh.restype = ctypes.c_double
    lib.forge_ref_num_threads.restype = i
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _configure(ctypes.CDLL(build()))
    return _lib


def use_library(path):
    """Points the binding at another build of the oracle (used by the tests that plant mistakes in a
    copy of the C source to see that the pins catch them).  ``None`` restores the real one."""
    global _lib
    _lib = None if path is None else _configure(ctypes.CDLL(path))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a):
    return a.ctypes.data_as(_dp)


def _lens_ptr(lens):
    if lens is None:
        return None, None
    l32 = np.ascontiguousarray(lens, dtype=np.int32)
    return l32, l32.ctypes.data_as(_ip)


def _check(status, what):
    if status != 0:
        raise ValueError(f"{what}: invalid argument (status {status})")


def attn(q, k, v, mask_kind=0, lens=None, scale=1.0):
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, Hq, Sq, D = q.shape
    _, Hkv, Skv, _ = k.shape
    assert k.shape == v.shape == (B, Hkv, Skv, D)
    out = np.empty_like(q)
    keep, lp = _lens_ptr(lens)
    _check(_load().forge_ref_attn(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, Hq, Hkv, Sq, Skv, D,
                                  int(mask_kind), lp, float(scale)), "forge_ref_attn")
    return out


def attn_probs(q, k, v, mask_kind=0, lens=None, scale=1.0):
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, Hq, Sq, D = q.shape
    _, Hkv, Skv, _ = k.shape
    assert k.shape == v.shape == (B, Hkv, Skv, D)
    out = np.empty_like(q)
    probs = np.empty((B, Hq, Sq, Skv), dtype=np.float64)
    keep, lp = _lens_ptr(lens)
    _check(_load().forge_ref_attn_probs(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(probs), B, Hq, Hkv,
                                        Sq, Skv, D, int(mask_kind), lp, float(scale)), "forge_ref_attn_probs")
    return out, probs


def attn_bias(q, k, v, bias, mask_kind=0, lens=None, scale=1.0, return_probs=False):
    """Attention with an additive bias [B, Hb, Sq, Skv] (Hb = 1 or Hq) on the scaled scores."""
    q, k, v, bias = _f64(q), _f64(k), _f64(v), _f64(bias)
    B, Hq, Sq, D = q.shape
    _, Hkv, Skv, _ = k.shape
    assert k.shape == v.shape == (B, Hkv, Skv, D)
    Hb = bias.shape[1]
    assert bias.shape == (B, Hb, Sq, Skv)
    out = np.empty_like(q)
    probs = np.empty((B, Hq, Sq, Skv), dtype=np.float64) if return_probs else None
    keep, lp = _lens_ptr(lens)
    _check(_load().forge_ref_attn_bias(_ptr(q), _ptr(k), _ptr(v), _ptr(out), None if probs is None else _ptr(probs),
                                       B, Hq, Hkv, Sq, Skv, D, int(mask_kind), lp, float(scale), _ptr(bias), Hb),
           "forge_ref_attn_bias")
    return (out, probs) if return_probs else out


def attn_decode(q, k_cache, v_cache, lens, scale=1.0):
    q, k_cache, v_cache = _f64(q), _f64(k_cache), _f64(v_cache)
    B, Hq, D = q.shape
    _, Hkv, Smax, _ = k_cache.shape
    assert k_cache.shape == v_cache.shape == (B, Hkv, Smax, D)
    out = np.empty_like(q)
    keep, lp = _lens_ptr(lens)
    _check(_load().forge_ref_attn_decode(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(out), B, Hq, Hkv,
                                         Smax, D, lp, float(scale)), "forge_ref_attn_decode")
    return out


def linear_bias_gelu(x, w, b):
    x, w, b = _f64(x), _f64(w), _f64(b)
    M, K = x.shape
    K2, N = w.shape
    assert K2 == K and b.shape == (N,)
    y = np.empty((M, N), dtype=np.float64)
    _check(_load().forge_ref_linear_bias_gelu(_ptr(x), _ptr(w), _ptr(b), _ptr(y), M, N, K),
           "forge_ref_linear_bias_gelu")
    return y


ACT_GELU_TANH, ACT_GELU_ERF, ACT_RELU, ACT_SILU, ACT_NONE = range(5)


def linear_act(x, w, b=None, residual=None, act=ACT_GELU_TANH, w_layout=0):
    """act(x W + b) + residual; w is [K,N] (w_layout 0) or [N,K] (w_layout 1); b, residual optional."""
    x, w = _f64(x), _f64(w)
    M, K = x.shape
    N = w.shape[1] if w_layout == 0 else w.shape[0]
    assert w.shape == ((K, N) if w_layout == 0 else (N, K))
    b = None if b is None else _f64(b)
    residual = None if residual is None else _f64(residual)
    assert b is None or b.shape == (N,)
    assert residual is None or residual.shape == (M, N)
    y = np.empty((M, N), dtype=np.float64)
    _check(_load().forge_ref_linear_act(_ptr(x), _ptr(w), None if b is None else _ptr(b),
                                        None if residual is None else _ptr(residual), _ptr(y), M, N, K,
                                        int(act), int(w_layout)), "forge_ref_linear_act")
    return y


def linear_w8(x, wq, scale, b=None, residual=None, act=ACT_GELU_TANH):
    """act(scale[n] * (x Wq^T)[m,n] + b) + residual; Wq [N,K] holds integers in [-128, 127]."""
    x, wq, scale = _f64(x), _f64(wq), _f64(scale)
    M, K = x.shape
    N = wq.shape[0]
    assert wq.shape == (N, K) and scale.shape == (N,)
    assert np.all(wq == np.round(wq)) and wq.min() >= -128 and wq.max() <= 127
    b = None if b is None else _f64(b)
    residual = None if residual is None else _f64(residual)
    y = np.empty((M, N), dtype=np.float64)
    _check(_load().forge_ref_linear_w8(_ptr(x), _ptr(wq), _ptr(scale), None if b is None else _ptr(b),
                                       None if residual is None else _ptr(residual), _ptr(y), M, N, K, int(act)),
           "forge_ref_linear_w8")
    return y


def linear_swiglu(x, wg, wu, w_layout=0):
    """silu(x Wg) * (x Wu); Wg, Wu are [K,N] (w_layout 0) or [N,K] (w_layout 1)."""
    x, wg, wu = _f64(x), _f64(wg), _f64(wu)
    M, K = x.shape
    N = wg.shape[1] if w_layout == 0 else wg.shape[0]
    assert wg.shape == wu.shape == ((K, N) if w_layout == 0 else (N, K))
    y = np.empty((M, N), dtype=np.float64)
    _check(_load().forge_ref_linear_swiglu(_ptr(x), _ptr(wg), _ptr(wu), _ptr(y), M, N, K, int(w_layout)),
           "forge_ref_linear_swiglu")
    return y


def gelu_tanh(z: float) -> float:
    return float(_load().forge_ref_gelu_tanh(float(z)))


def num_threads() -> int:
    return int(_load().forge_ref_num_threads())
