"""GPU parity: absmean ternary quantizer (Eq. 1-2) and the 2-bit format vs the oracle."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,K", [(16, 128), (512, 512), (2048, 2048), (528, 384), (2048, 8192)])
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
