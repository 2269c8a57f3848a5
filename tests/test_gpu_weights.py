"""GPU parity: absmean ternary quantizer (Eq. 1-2) and the 2-bit format vs the oracle."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,K", [(16, 128), (512, 512), (2048, 2048), (528, 384), (2048, 8192), (16, 32768), (1040, 1152)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_weight_quant_is_bit_exact(N, K, dtype):
    W = wl.rows("latent", 11, N + K, K, 0, N, dtype)
    Wd = torch.from_numpy(W).cuda()
    if dtype == "bf16":
        Wd = Wd.to(torch.bfloat16)
    packed, alpha = hbl.hbl_quantize_weights(Wd, EPS)
    wt, a = orc.weight_quant(W, EPS, 32)
    assert alpha.cpu().numpy()[0] == a
    got = hbl.hbl_unpack_weights(packed, N, K).cpu().numpy()
    assert np.array_equal(got, wt)


def test_packed_format_is_the_documented_one():
    """Decode the packed bytes on the host exactly as include/hbl.h describes them."""
    N, K = 32, 256
    W = wl.rows("latent", 3, 77, K, 0, N, "f32")
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    words = packed.cpu().numpy().view(np.uint32).reshape((N + 127) // 128, K // 128, 2, 128, 4)
    wt, _ = orc.weight_quant(W, EPS, 32)
    dec = np.zeros((N, K), np.int8)
    for rb in range(words.shape[0]):
        for kb in range(K // 128):
            for h in range(2):
                for row in range(128):
                    R = 128 * rb + row
                    for v in range(4):
                        w = int(words[rb, kb, h, row, v])
                        for i in range(4):
                            for b in range(4):
                                u = (w >> (8 * b + 2 * i)) & 3
                                if R < N:
                                    dec[R, 128 * kb + 16 * (4 * h + v) + 4 * i + b] = u - 1
                                else:
                                    assert u == 1          # padding rows are zeros
    assert np.array_equal(dec, wt)
    assert packed.numel() == ((N + 127) // 128) * 128 * K // 4


def test_weight_quant_special_values():
    N, K = 16, 128
    W = np.zeros((N, K), np.float32)
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    assert alpha.item() == 0.0
    assert np.all(hbl.hbl_unpack_weights(packed, N, K).cpu().numpy() == 0)
    W[:] = 0.5; W[0, :] = -0.5; W[1, 0] = 100.0
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    wt, a = orc.weight_quant(W, EPS, 32)
    assert alpha.item() == a
    assert np.array_equal(hbl.hbl_unpack_weights(packed, N, K).cpu().numpy(), wt)


def _signs(shape, seed):
    return np.where(np.random.default_rng(seed).integers(0, 2, size=shape) == 1, 1.0, -1.0)


@pytest.mark.parametrize("k", [1, 2, 77, 4095, 0x3FFFFF])
def test_weight_quant_decisions_next_to_the_threshold_f32(k):
    """Eq. 1-2 round W / (alpha + eps) half to even: the result changes exactly where the fp32 quotient passes
    1/2.  The tensor is built so that alpha is known exactly (every group of four entries adds up to 4 a in
    magnitude), d = alpha + eps = 1 + k 2^-23, and the first entry of each group sits on d / 2 or a few fp32
    steps beside it; the oracle decides by the fp32 division."""
    N, K = 16, 128
    eps = 2.0 ** -17
    d = 1.0 + k * 2.0 ** -23
    a = d - eps
    h = d / 2
    mag = np.full(N * K, a)
    steps = np.arange(N * K // 4) % 9 - 4                          # -4 .. 4 fp32 steps (2^-24) beside d / 2
    x = h + steps * 2.0 ** -24
    mag[0::4] = x
    mag[1::4] = 0.75 - x
    mag[2::4] = mag[3::4] = (4 * a - 0.75) / 2
    assert np.array_equal(mag.astype(np.float32).astype(np.float64), mag)      # all exactly fp32
    assert np.float32(np.float32(a) + np.float32(eps)) == np.float32(d)
    W = (mag * _signs(mag.shape, k)).astype(np.float32).reshape(N, K)
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), eps)
    wt, al = orc.weight_quant(W, eps, 32)
    assert al == np.float32(a) and alpha.item() == al
    got = hbl.hbl_unpack_weights(packed, N, K).cpu().numpy()
    assert np.array_equal(got, wt)
    on_or_below = np.abs(W.reshape(-1)[0::4]) <= np.float32(h)                   # what the rounding rule implies
    assert np.array_equal(wt.reshape(-1)[0::4] == 0, on_or_below)


@pytest.mark.parametrize("eps", [2.0 ** -9, 2.0 ** -8, 3 * 2.0 ** -10, 1e-5, 2.0 ** -8 + 2.0 ** -20])
def test_weight_quant_decisions_next_to_the_threshold_bf16(eps):
    """The same for bf16 latents: alpha = 1/2 exactly, d / 2 = 1/4 + eps / 2 falls on or between bf16 values."""
    N, K = 16, 384
    mag = np.full(N * K, 0.5)
    m = np.arange(N * K // 3) % 6 - 2                               # -2 .. 3 bf16 steps (2^-9) beside 1/4
    mag[0::3] = 0.25 + m * 2.0 ** -9
    mag[1::3] = 0.125 - m * 2.0 ** -9
    mag[2::3] = 1.125
    Wt = torch.from_numpy((mag * _signs(mag.shape, 5)).reshape(N, K)).to(torch.bfloat16)
    W = Wt.float().numpy()
    assert np.array_equal(np.abs(W.reshape(-1)).astype(np.float64), mag)         # all exactly bf16
    packed, alpha = hbl.hbl_quantize_weights(Wt.cuda(), eps)
    wt, al = orc.weight_quant(W, eps, 32)
    assert al == 0.5 and alpha.item() == 0.5
    assert np.array_equal(hbl.hbl_unpack_weights(packed, N, K).cpu().numpy(), wt)
    half_d = np.float32(np.float32(0.5) + np.float32(eps)) / np.float32(2)
    assert np.array_equal(wt.reshape(-1)[0::3] == 0, np.abs(W.reshape(-1)[0::3]) <= half_d)


@pytest.mark.parametrize("N,K,dtype", [(144, 512, "f32"), (528, 2048, "f32"), (256, 8192, "bf16"), (2048, 4096, "f32")])
def test_rotated_weight_quant(N, K, dtype):
    """Weight-and-activation rotation (the ablation's other variant): W H is ternarised instead of W.
    Two stages, each against the oracle: the transformed rows (fp32 butterflies vs the fp64 transform), then
    Eq. 1-2 on exactly the fp32 values the kernel produced (bit-exact, as for the plain weights) -- the ternary
    decision is taken on the same numbers on both sides."""
    import torch
    from oracle import hbl_oracle as orc
    W = wl.rows("latent", 60 + N, 7, K, 0, N, dtype)
    Wd = torch.from_numpy(W).cuda()
    if dtype == "bf16":
        Wd = Wd.bfloat16()
    packed, alpha = hbl.hbl_quantize_weights_rotated(Wd, EPS)
    assert hbl.hbl_check_status() == 0
    Wr = hbl.hbl_hadamard_f32(Wd)
    want = orc.hadamard(W)
    assert np.all(np.abs(Wr.cpu().numpy() - want) <= 1e-5 * np.abs(want).max(axis=1, keepdims=True))
    wt, al = orc.weight_quant(Wr.cpu().numpy(), EPS, 32)
    assert alpha.item() == al
    assert np.array_equal(hbl.hbl_unpack_weights(packed, N, K).cpu().numpy(), wt)
    # the same as the two public steps one after the other
    p2, a2 = hbl.hbl_quantize_weights(Wr, EPS)
    assert torch.equal(packed, p2) and torch.equal(alpha, a2)


def test_rotated_weights_in_the_layer():
    """With both sides rotated the layer still approximates W x: (W H)(H x) = W x before quantization."""
    import torch
    from oracle import hbl_oracle as orc
    from parity_utils import check_y, oracle_layer, to_dev
    N, K, T = 272, 2048, 24
    W = wl.rows("latent", 71, 7, K, 0, N, "f32")
    x = wl.rows("attn_out", 71, 1, K, 0, T, "bf16")
    Wd = torch.from_numpy(W).cuda()
    packed, alpha = hbl.hbl_quantize_weights_rotated(Wd, EPS)
    y = hbl.hbl_forward(to_dev(x, "bf16"), packed, alpha, N, 8, True, EPS)
    o = oracle_layer(x, hbl.hbl_hadamard_f32(Wd).cpu().numpy(), 8, True)      # the oracle's layer on the rotated latents
    check_y(y, o["y64"])
    dense = x.astype(np.float64) @ W.astype(np.float64).T
    yf = y.float().cpu().numpy().astype(np.float64)
    corr = (yf * dense).sum() / np.sqrt((yf ** 2).sum() * (dense ** 2).sum())
    assert corr > 0.8                                                          # ternary weights: a coarse but aligned product
