"""GPU parity: the integer contraction of Eq. 7, both kernels, bit-exact given identical codes."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS

pytestmark = pytest.mark.gpu


def setup(T, K, N, bits, seed):
    rng = np.random.default_rng(seed)
    lo, hi = (-128, 128) if bits == 8 else (-8, 8)
    q = rng.integers(lo, hi, size=(T, K), dtype=np.int8)
    W = wl.rows("latent", seed, 50, K, 0, N, "f32")
    packed, _ = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    wt, _ = orc.weight_quant(W, EPS, 32)
    return q, packed, wt


@pytest.mark.parametrize("T,K,N", [(1, 128, 16), (3, 384, 144), (8, 2048, 2048), (16, 8192, 2048),
                                   (17, 512, 528), (33, 4096, 1024), (64, 1024, 4096), (5, 16384, 256),
                                   (100, 2048, 784), (128, 4096, 2048), (65, 384, 4112), (300, 1024, 528), (512, 2048, 256)])
@pytest.mark.parametrize("bits", [4, 8])
def test_stream_kernel_bit_exact(T, K, N, bits):
    q, packed, wt = setup(T, K, N, bits, T * 1000 + K + N)
    qd = torch.from_numpy(q).cuda()
    csum = qd.to(torch.int32).sum(1, dtype=torch.int32)
    got = hbl.hbl_gemm_i32(qd, csum, packed, N, hbl.PATH_STREAM).cpu().numpy()
    assert np.array_equal(got, orc.gemm(q, wt))


@pytest.mark.parametrize("T,K,N", [(1, 128, 16), (128, 128, 256), (300, 512, 528), (129, 1024, 2048),
                                   (1000, 2048, 272), (64, 8192, 512), (260, 16384, 256)])
@pytest.mark.parametrize("bits", [4, 8])
def test_tensor_kernel_bit_exact(T, K, N, bits):
    q, packed, wt = setup(T, K, N, bits, T * 1000 + K + N + 1)
    got = hbl.hbl_gemm_i32(torch.from_numpy(q).cuda(), None, packed, N, hbl.PATH_TENSOR).cpu().numpy()
    assert hbl.hbl_check_status() == 0
    assert np.array_equal(got, orc.gemm(q, wt))


def test_extreme_codes_do_not_overflow():
    K, N, T = 16384, 256, 130
    q = np.full((T, K), -128, np.int8)
    W = np.full((N, K), -1.0, np.float32)
    packed, _ = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    got = hbl.hbl_gemm_i32(torch.from_numpy(q).cuda(), None, packed, N, hbl.PATH_TENSOR).cpu().numpy()
    assert np.all(got == 128 * K)
    qs = torch.from_numpy(q[:16]).cuda()
    got = hbl.hbl_gemm_i32(qs, qs.to(torch.int32).sum(1, dtype=torch.int32), packed, N, hbl.PATH_STREAM).cpu().numpy()
    assert np.all(got == 128 * K)


@pytest.mark.parametrize("T", [16, 100])
def test_stream_kernel_largest_accumulators(T):
    """The small-batch kernel feeds the tensor core 64 (w + 1), so its accumulators are 64 times the sums of
    Eq. 7 plus 64 times the code sums: the largest they can get is at the longest row the library accepts,
    all weights +1 and all codes -128 (or 127)."""
    K, N = 32768, 144
    W = np.full((N, K), 1.0, np.float32)
    packed, _ = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    q = np.full((T, K), -128, np.int8)
    q[1::2] = 127
    qd = torch.from_numpy(q).cuda()
    got = hbl.hbl_gemm_i32(qd, qd.to(torch.int32).sum(1, dtype=torch.int32), packed, N, hbl.PATH_STREAM).cpu().numpy()
    assert hbl.hbl_check_status() == 0
    want = q.astype(np.int64).sum(1, keepdims=True).repeat(N, 1)
    assert np.array_equal(got, want)


def test_both_kernels_agree_and_runs_are_deterministic():
    T, K, N = 48, 4096, 4096
    q, packed, wt = setup(T, K, N, 4, 99)
    qd = torch.from_numpy(q).cuda()
    csum = qd.to(torch.int32).sum(1, dtype=torch.int32)
    a = hbl.hbl_gemm_i32(qd, csum, packed, N, hbl.PATH_STREAM)
    b = hbl.hbl_gemm_i32(qd, None, packed, N, hbl.PATH_TENSOR)
    c = hbl.hbl_gemm_i32(qd, csum, packed, N, hbl.PATH_STREAM)
    assert torch.equal(a, b) and torch.equal(a, c)
