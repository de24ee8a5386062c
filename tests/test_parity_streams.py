"""GPU: calls issued on two streams at once give the same bits as the same calls issued one after the other.
The library keeps no state between calls except the error word; every kernel is launched with programmatic
stream serialisation and waits for its predecessor in its own stream only, so streams must not disturb each
other (each decode call has its own workspace)."""
import numpy as np
import pytest
import torch

from paper_2604_16498_b200 import binding, workloads as wl
from util import to_device

pytestmark = pytest.mark.gpu


def test_two_streams_give_the_serial_results():
    att = wl.attention_workload("t", 81, 2, 8, 2, 700, 700, 128, wl.MASK_CAUSAL, 128 ** -0.5, "bf16")
    lin = wl.linear_workload("t", 82, 1024, 768, 512, w_std=512 ** -0.5, b_std=0.5)
    dec = wl.decode_workload("t", 83, 8, 16, 4, 2048, 128, 8, 128 ** -0.5, (200, 2048))
    q, k, v = to_device(att.q), to_device(att.k), to_device(att.v)
    x, w, b = to_device(lin.x), to_device(lin.w), to_device(lin.b)
    dq, kc, vc = to_device(dec.q), to_device(dec.k_cache), to_device(dec.v_cache)
    lens = torch.from_numpy(dec.lens).cuda()
    nbytes = binding.attn_decode_workspace_bytes(dec.B, dec.Hq, dec.D, dec.num_splits)

    def work(ws):
        outs = []
        for _ in range(3):
            outs.append(binding.attn_fused(q, k, v, att.mask_kind, None, att.scale))
            outs.append(binding.linear_bias_gelu(x, w, b))
            outs.append(binding.attn_decode_splitkv(dq, kc, vc, lens, dec.num_splits, dec.scale, workspace=ws))
        return outs

    serial = work(torch.zeros(nbytes, dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    ws1 = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")  # the arrival counters start at zero
    ws2 = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(s1):
        a = work(ws1)
    with torch.cuda.stream(s2):
        c = work(ws2)
    torch.cuda.synchronize()
    binding.check_status()
    for got in (a, c):
        for g, want in zip(got, serial):
            assert torch.equal(g, want)
