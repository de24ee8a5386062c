"""Helpers shared by the GPU parity tests: moving seeded inputs to the device and the
tolerances (fp32: max-abs 1e-4; bf16 in / fp32 accumulate: max-abs 2e-2 and mean-abs 2e-3
on unit-variance data)."""
import numpy as np
import torch

F32_MAX_ABS = 1e-4
BF16_MAX_ABS = 2e-2
BF16_MEAN_ABS = 2e-3


def to_device(t):
    """workloads.Tensor -> CUDA tensor holding exactly the same values."""
    if t.dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(t.device_bits)).cuda()
    if t.dtype == "f16":
        return torch.from_numpy(np.ascontiguousarray(t.device_bits).view(np.float16)).cuda()
    return torch.from_numpy(np.ascontiguousarray(t.device_bits).view(np.int16)).view(torch.bfloat16).cuda()


def to_pinned(t):
    if t.dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(t.device_bits)).pin_memory()
    return torch.from_numpy(np.ascontiguousarray(t.device_bits).view(np.int16)).view(torch.bfloat16).pin_memory()


def bf16_tensor(values_f64):
    """fp64 numpy array of bf16-representable values -> CUDA bf16 tensor."""
    return torch.from_numpy(np.asarray(values_f64, dtype=np.float32)).to(torch.bfloat16).cuda()


def to_f64(x: torch.Tensor) -> np.ndarray:
    return x.detach().float().cpu().double().numpy()


def assert_close_f32(got, ref):
    err = np.abs(to_f64(got) - ref)
    assert np.isfinite(to_f64(got)).all()
    assert err.max() <= F32_MAX_ABS, f"max-abs {err.max():.3e} > {F32_MAX_ABS}"


def assert_close_bf16(got, ref):
    g = to_f64(got)
    assert np.isfinite(g).all()
    err = np.abs(g - ref)
    assert err.max() <= BF16_MAX_ABS, f"max-abs {err.max():.3e} > {BF16_MAX_ABS}"
    assert err.mean() <= BF16_MEAN_ABS, f"mean-abs {err.mean():.3e} > {BF16_MEAN_ABS}"
    return err.max(), err.mean()


# ---- canary-guarded buffers: outputs and workspaces carved out of a larger allocation filled with a
# sentinel, so that a write outside the buffer (a clipped TMA store that did not clip, a ragged tail
# stored with full-width vectors) shows up even when the result itself is right.
GUARD_BYTES = 4096
_SENTINEL = 0x5A


class Guarded:
    """A CUDA tensor of `shape` / `dtype` with GUARD_BYTES of sentinel on both sides."""

    def __init__(self, shape, dtype, fill_nan=True):
        es = torch.empty((), dtype=dtype).element_size()
        n = int(np.prod(shape)) * es
        self.nbytes = n
        self.raw = torch.full((GUARD_BYTES + n + GUARD_BYTES,), _SENTINEL, dtype=torch.uint8, device="cuda")
        assert self.raw.data_ptr() % 256 == 0
        self.tensor = self.raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)
        if fill_nan and dtype in (torch.bfloat16, torch.float16, torch.float32):
            self.tensor.fill_(float("nan"))  # a position the kernel fails to write stays visible

    def assert_intact(self):
        torch.cuda.synchronize()
        lo = self.raw[:GUARD_BYTES]
        hi = self.raw[GUARD_BYTES + self.nbytes:]
        assert bool((lo == _SENTINEL).all()), "bytes before the buffer were overwritten"
        assert bool((hi == _SENTINEL).all()), "bytes after the buffer were overwritten"
