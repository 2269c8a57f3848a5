"""GPU parity: the low-bit attention-state quantizer (section 3.1) vs the oracle.

The statistic (a maximum of bf16 values) is exact on both sides and both take the rounding decision in IEEE fp32
in the same order, so codes and scales must agree bit for bit; the packed bytes are decoded here, on the host,
from the layout the header documents."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl

pytestmark = pytest.mark.gpu
EPS = 1e-5


def decode(packed: np.ndarray, bits: int, D: int) -> np.ndarray:
    """[R, D*bits/8] bytes -> [R, D] codes: element d is the bits [bits*d, bits*d+bits) of the row's little-endian bit string."""
    R = packed.shape[0]
    bitstr = np.unpackbits(packed, axis=1, bitorder="little").reshape(R, D, bits)
    return (bitstr.astype(np.int32) << np.arange(bits)).sum(axis=2).astype(np.uint8)


def states(T, H, D, seed, kind="gauss"):
    return wl.rows(kind, seed, 40, H * D, 0, T, "bf16").reshape(T, H, D)


@pytest.mark.parametrize("bits", [3, 4, 8])
@pytest.mark.parametrize("T,H,D", [(1, 1, 64), (37, 5, 128), (130, 32, 128), (9, 3, 256), (257, 8, 64)])
def test_kv_codes_and_scales_match_oracle(bits, T, H, D):
    x = states(T, H, D, 500 + bits + T)
    x[T // 2, 0, :] = 0                                            # an all-zero head
    codes, scale, _, _ = hbl.hbl_quantize_kv(torch.from_numpy(x).cuda().bfloat16(), bits, 0, EPS)
    assert hbl.hbl_check_status() == 0
    u, v, s = orc.kv_quant(x.reshape(T * H, D), bits, EPS, 32)
    assert np.array_equal(decode(codes.cpu().numpy(), bits, D), u)
    assert np.array_equal(scale.cpu().numpy(), s.astype(np.float32))
    # and against the formula taken in fp64: a code may differ by one only next to a rounding boundary
    u64, v64, _ = orc.kv_quant(x.reshape(T * H, D), bits, EPS, 64)
    diff = u.astype(np.int32) - u64.astype(np.int32)
    bad = np.nonzero(diff)
    assert len(bad[0]) <= max(1, int(1e-4 * u.size)) and np.all(np.abs(diff[bad]) == 1)
    if len(bad[0]):
        b = u64[bad].astype(np.float64) - (1 << (bits - 1)) + 0.5 * diff[bad]
        assert np.all(np.abs(v64[bad] - b) <= 1e-5 * np.maximum(1.0, np.abs(b)))


@pytest.mark.parametrize("bits", [3, 4])
def test_kv_bos_rows_kept_at_8_bits(bits):
    T, H, D, S = 200, 4, 128, 64                                   # 4 sequences, the last one ragged
    x = states(T, H, D, 600 + bits, "attn_out")
    codes, scale, bos_codes, bos_scale = hbl.hbl_quantize_kv(torch.from_numpy(x).cuda().bfloat16(), bits, S, EPS)
    assert hbl.hbl_check_status() == 0
    u, _, s = orc.kv_quant(x.reshape(T * H, D), bits, EPS, 32)
    assert np.array_equal(decode(codes.cpu().numpy(), bits, D), u)  # the low-bit array covers every token
    bos = x[::S].reshape(-1, D)                                    # tokens 0, 64, 128, 192
    u8, _, s8 = orc.kv_quant(bos, 8, EPS, 32)
    assert np.array_equal(bos_codes.cpu().numpy().reshape(-1, D), u8)
    assert np.array_equal(bos_scale.cpu().numpy(), s8.astype(np.float32))
    # the same through the oracle's per-row widths: [BOS] rows at 8, the rest at `bits`
    br = np.where((np.arange(T) % S == 0)[:, None], 8, bits).repeat(H, axis=1).reshape(-1).astype(np.int32)
    um, _, sm = orc.kv_quant(x.reshape(T * H, D), bits, EPS, 32, bits_row=br)
    assert np.array_equal(um[br == 8], u8) and np.array_equal(um[br != 8], u[br != 8])


def test_kv_dequantization_error_and_extremes():
    T, H, D = 64, 8, 128
    x = states(T, H, D, 700, "attn_out")
    for bits in (3, 4, 8):
        codes, scale, _, _ = hbl.hbl_quantize_kv(torch.from_numpy(x).cuda().bfloat16(), bits, 0, EPS)
        u = decode(codes.cpu().numpy(), bits, D).astype(np.float64)
        half = 1 << (bits - 1)
        s = scale.cpu().numpy().astype(np.float64)
        assert u.min() >= 1 and u.max() == 2 * half - 1
        err = np.abs((u - half) * s[:, None] - x.reshape(-1, D))
        assert np.all(err <= 0.5 * s[:, None] * (1 + 1e-6) + 3e-5 * np.abs(x.reshape(-1, D)).max(1, keepdims=True))


def test_kv_zero_tokens_and_full_size():
    out = hbl.hbl_quantize_kv(torch.empty((0, 8, 128), dtype=torch.bfloat16, device="cuda"), 4)
    assert out[0].shape[0] == 0
    # the 7B shape (32 heads of 128) at 16384 tokens, sampled rows recomputed by the oracle
    T, H, D = 16384, 32, 128
    rows = states(4096, H, D, 800)
    xd = torch.from_numpy(rows).cuda().bfloat16().repeat(4, 1, 1)
    codes, scale, bos_codes, bos_scale = hbl.hbl_quantize_kv(xd, 3, 2048, EPS)
    assert hbl.hbl_check_status() == 0
    toks = [0, 1, 2047, 2048, 4095, 4096, 9999, T - 1]
    ref = np.stack([rows[t % 4096] for t in toks]).reshape(-1, D)
    u, _, s = orc.kv_quant(ref, 3, EPS, 32)
    idx = np.concatenate([np.arange(t * H, (t + 1) * H) for t in toks])
    assert np.array_equal(decode(codes[idx].cpu().numpy(), 3, D), u)
    assert np.array_equal(scale[idx].cpu().numpy(), s.astype(np.float32))
    assert torch.equal(codes[: 4096 * H], codes[4096 * H: 8192 * H])
    u8, _, s8 = orc.kv_quant(rows[2048].reshape(-1, D), 8, EPS, 32)   # token 2048 opens the second sequence
    assert np.array_equal(bos_codes[1].cpu().numpy().reshape(-1, D), u8)
