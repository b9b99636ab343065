"""The fp8 (e4m3, power-of-two scale per page and KV head) copy of a workload's cache: what the bytes stand
for is exactly representable in bf16, is the nearest e4m3 value of the scaled input, and uses the smallest
scale that fits the block - so the oracle, run on the dequantised bf16 cache, is the reference of the fp8
path without any change."""
import numpy as np
import torch

from workloads import WorkloadSpec, make_workload, quantize_kv_fp8


def _w():
    return make_workload(WorkloadSpec(name="q8", config=9, batch=2, n_q_heads=8, n_kv_heads=2, P=4, K_c=24,
                                      seq_lens=(300, 177), needles=3, needle_positions="uniform"), seed=5)


def _decode_e4m3(byte: int) -> float:
    """the format's definition (OCP e4m3fn): 1 sign, 4 exponent (bias 7), 3 mantissa bits, no infinities"""
    s, e, m = byte >> 7, (byte >> 3) & 15, byte & 7
    v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return -v if s else v


def test_bytes_scales_and_dequantised_values_agree():
    w = _w()
    wq, k8, v8, ke, ve = quantize_kv_fp8(w)
    table = torch.tensor([_decode_e4m3(b) if (b & 0x7f) != 0x7f else float("nan") for b in range(256)])
    for raw, ex, deq, src in ((k8, ke, wq.k_cache, w.k_cache), (v8, ve, wq.v_cache, w.v_cache)):
        assert raw.dtype == torch.uint8 and ex.dtype == torch.int8 and deq.dtype == torch.bfloat16
        assert not ((raw & 0x7f) == 0x7f).any()                              # no NaN encodings
        vals = table[raw.long()] * torch.exp2(ex.float())[:, :, None, None]
        assert torch.equal(vals, deq.float())                                # bytes * 2^e == the bf16 cache, exactly
        x = src.float()
        amax = x.abs().amax(dim=(2, 3))
        used = amax > 0
        # the smallest power of two that fits: the block fits, and half the scale would not
        assert (amax[used] / torch.exp2(ex.float()[used]) <= 448.0).all()
        assert (amax[used] / torch.exp2(ex.float()[used] - 1) > 448.0).all()
        # nearest e4m3: relative error at most 2^-4 for values in the normal range of the scaled block
        scaled = (x / torch.exp2(ex.float())[:, :, None, None]).abs()
        normal = scaled >= 2.0 ** -6
        err = (deq.float() - x).abs()
        assert (err[normal] <= x.abs()[normal] * 2.0 ** -4).all()
        assert (err[~normal] <= torch.exp2(ex.float())[:, :, None, None].expand_as(err)[~normal] * 2.0 ** -10).all()
    # everything else is the same workload
    assert torch.equal(wq.q, w.q) and torch.equal(wq.block_table, w.block_table) and torch.equal(wq.seq_lens, w.seq_lens)
