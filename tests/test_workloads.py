"""The seeded input generators: reproducible, correctly distributed, exactly representable."""
import numpy as np
import torch

from paper_2604_16498_b200 import workloads as wl


def test_splitmix64_published_vectors():
    # First outputs of the splitmix64 reference generator seeded with 0 (widely published test vector).
    got = wl.splitmix64(0, 3)
    assert [int(x) for x in got] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    assert (wl.splitmix64(0, 5, start=2) == wl.splitmix64(0, 7)[2:]).all()


def test_normal_moments_and_reproducibility():
    x = wl.normal_f64(123, 400_001)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert abs((x ** 3).mean()) < 0.03 and abs((x ** 4).mean() - 3.0) < 0.1
    assert (wl.normal_f64(123, 400_001) == x).all()
    assert (wl.normal_f64(123, 1001) == x[:1001]).all()
    y = wl.normal_f64(9, 100_000, std=0.02)
    assert abs(y.std() - 0.02) < 0.0005


def test_bf16_rounding_matches_torch_rne():
    x32 = wl.normal_f64(5, 100_000).astype(np.float32)
    x32[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]   # exact ties: to even
    bits = wl.f32_to_bf16_bits(x32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (bits == ref).all()
    wide = wl.bf16_bits_to_f64(bits)
    assert (wide == torch.from_numpy(x32).to(torch.bfloat16).double().numpy()).all()


def test_uniform_int_bounds_inclusive():
    v = wl.uniform_int(77, 20_000, 16, 128)
    assert v.min() == 16 and v.max() == 128 and v.dtype == np.int32


def test_config_shapes_and_counts():
    c1 = wl.cfg1_gpt2_f32()
    assert c1.q.values.shape == (1, 12, 128, 64) and c1.q.device_bits.dtype == np.float32
    assert c1.flops() == 25_362_432 and c1.bytes() == 1_572_864
    c3 = wl.cfg3_encoder()
    assert c3.lens.min() >= 16 and c3.lens.max() <= 128
    assert c3.flops() == 393_216 * int(c3.lens.sum())
    assert c3.bytes() == 12_582_912 + 3_072 * int(c3.lens.sum())
    lw = wl.cfg2_linear(M=64)
    assert lw.w.values.shape == (768, 3072) and abs(lw.w.values.std() - 0.02) < 1e-3
    assert lw.flops() * (8192 // 64) == 38_654_705_664
    c2 = wl.cfg2_attention(B=1)
    assert c2.flops() * 8 == 12_897_484_800 and c2.bytes() * 8 == 50_331_648


def test_f16_rounding_matches_torch_rne():
    """The fp16 tensors hold exactly what torch's fp32 -> fp16 conversion (round to nearest even) gives, and
    the oracle's values are the exact widening of the patterns the GPU reads."""
    t = wl.normal_tensor(77, (4096,), "f16")
    x32 = wl.normal_f64(77, 4096).astype(np.float32)
    ref = torch.from_numpy(x32).to(torch.float16)
    assert np.array_equal(t.device_bits, ref.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(t.values, ref.double().numpy())
