"""Host-only checks of the C ABI: the library builds, loads without a GPU, exports every
function that include/forge.h declares, and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

from paper_2604_16498_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "forge.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(forge_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = _declared_functions()
    for must in ["forge_attn_fused", "forge_attn_fused_f32", "forge_attn_decode_splitkv",
                 "forge_attn_decode_workspace_bytes", "forge_linear_bias_gelu", "forge_check_status",
                 "forge_status_string", "forge_last_cuda_error"]:
        assert must in names


def test_every_declared_symbol_is_exported_and_bound(lib):
    for name in _declared_functions():
        assert hasattr(lib, name), f"{name} declared in forge.h but not exported by libforge.so"
        assert name in binding.SIGNATURES, f"{name} has no ctypes signature in the binding"


def test_status_strings(lib):
    assert lib.forge_status_string(0) == b"FORGE_OK"
    assert lib.forge_status_string(5) == b"FORGE_ERR_TIMEOUT"
    assert lib.forge_status_string(99) == b"FORGE_ERR_UNKNOWN"


def test_workspace_size(lib):
    # arrival counters (1088 KiB, or 68 bytes per (batch, head) if that is more) + num_splits partial slots per (batch, head)
    assert lib.forge_attn_decode_workspace_bytes(16, 32, 128, 16) == 17 * 65536 + 16 * 32 * 16 * (128 + 2) * 4
    assert lib.forge_attn_decode_workspace_bytes(3, 8, 40, 5) == 17 * 65536 + 3 * 8 * 5 * (64 + 2) * 4
    assert lib.forge_attn_decode_workspace_bytes(1024, 32, 128, 1) == 68 * 1024 * 32 + 1024 * 32 * (128 + 2) * 4
    assert lib.forge_attn_decode_workspace_bytes(4096, 8, 64, 1) == 4096 * 8 * 68 + 4096 * 8 * (64 + 2) * 4
    assert lib.forge_attn_decode_workspace_bytes(0, 32, 128, 16) == 0


P = 0x10000  # a fake, 16-byte aligned pointer: validation must reject the call before touching it


@pytest.mark.parametrize("fn", ["forge_attn_fused", "forge_attn_fused_f32"])
def test_attention_argument_validation(lib, fn):
    f = getattr(lib, fn)
    ok = dict(q=P, k=P, v=P, out=P, B=1, Hq=4, Hkv=2, Sq=8, Skv=8, D=64, mask=0, lens=None, scale=1.0, stream=None)

    def call(**kw):
        a = {**ok, **kw}
        return f(a["q"], a["k"], a["v"], a["out"], a["B"], a["Hq"], a["Hkv"], a["Sq"], a["Skv"], a["D"],
                 a["mask"], a["lens"], a["scale"], a["stream"])

    assert call(q=None) == binding.ERR_INVALID_ARG
    assert call(out=None) == binding.ERR_INVALID_ARG
    assert call(B=0) == binding.ERR_INVALID_ARG
    assert call(Sq=-1) == binding.ERR_INVALID_ARG
    assert call(Hq=3) == binding.ERR_INVALID_ARG          # Hq % Hkv != 0
    assert call(mask=4) == binding.ERR_INVALID_ARG
    assert call(mask=2) == binding.ERR_INVALID_ARG        # padding mask without lens
    assert call(k=P + 8) == binding.ERR_INVALID_ARG       # misaligned
    assert call(D=264) == binding.ERR_UNSUPPORTED         # beyond the largest head size
    if fn == "forge_attn_fused_f32":
        assert call(D=256) == binding.ERR_UNSUPPORTED     # the fp32 kernel has 64 and 128 only
    assert call(D=100) == binding.ERR_UNSUPPORTED         # rows are not multiples of 16 bytes


def test_decode_argument_validation(lib):
    f = lib.forge_attn_decode_splitkv
    need = lib.forge_attn_decode_workspace_bytes(2, 8, 128, 4)
    ok = dict(q=P, k=P, v=P, out=P, B=2, Hq=8, Hkv=2, Smax=64, D=128, lens=P, splits=4, scale=1.0, ws=P,
              wsb=need, stream=None)

    def call(**kw):
        a = {**ok, **kw}
        return f(a["q"], a["k"], a["v"], a["out"], a["B"], a["Hq"], a["Hkv"], a["Smax"], a["D"], a["lens"],
                 a["splits"], a["scale"], a["ws"], a["wsb"], a["stream"])

    assert call(lens=None) == binding.ERR_INVALID_ARG
    assert call(splits=0) == binding.ERR_INVALID_ARG
    assert call(splits=257) == binding.ERR_UNSUPPORTED
    assert call(ws=None) == binding.ERR_INVALID_ARG
    assert call(wsb=need - 1) == binding.ERR_WORKSPACE
    assert call(Hq=18, Hkv=2, wsb=1 << 30) == binding.ERR_UNSUPPORTED   # group size 9
    assert call(D=136) == binding.ERR_UNSUPPORTED
    assert call(D=100) == binding.ERR_UNSUPPORTED


def test_linear_argument_validation(lib):
    f = lib.forge_linear_bias_gelu
    assert f(None, P, P, P, 8, 8, 8, None) == binding.ERR_INVALID_ARG
    assert f(P, P, P, P, 0, 8, 8, None) == binding.ERR_INVALID_ARG
    assert f(P, P + 2, P, P, 8, 8, 8, None) == binding.ERR_INVALID_ARG
    assert f(P, P, P, P, 8, 12, 8, None) == binding.ERR_UNSUPPORTED   # N not a multiple of 8
    assert f(P, P, P, P, 8, 8, 20, None) == binding.ERR_UNSUPPORTED   # K not a multiple of 8


def test_host_variant_validation(lib):
    assert lib.forge_linear_bias_gelu_host(P, P, P, P, 8, 8, 8, None, 0, None) == binding.ERR_INVALID_ARG
    assert lib.forge_linear_bias_gelu_host(P, P, P, P, 8, 8, 8, 0x10000, 16, None) == binding.ERR_WORKSPACE
    assert lib.forge_attn_fused_host(P, P, P, P, 1, 2, 2, 8, 8, 64, 0, None, 1.0, 0x10000, 16, None) \
        == binding.ERR_WORKSPACE
    assert lib.forge_linear_host_scratch_bytes(128, 256, 64) >= 2 * (128 * 64 + 64 * 256 + 256 + 128 * 256)
