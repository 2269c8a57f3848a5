"""GPU parity: transform (Eq. 3-4) and activation quantizers (Eq. 5-6) vs the oracle."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS, check_codes, to_dev

pytestmark = pytest.mark.gpu

ALL_K = [128, 256, 512, 1024, 2048, 4096, 8192, 16384, 32768]


def make_x(K, T, seed, kind="attn_out", dtype="bf16"):
    return wl.rows(kind, seed, 1, K, 0, T, dtype)


@pytest.mark.parametrize("K", ALL_K)
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_hadamard_matches_oracle(K, dtype):
    T = 37 if K <= 8192 else 9           # ragged against every tokens-per-CTA grouping
    x = make_x(K, T, 100 + K, dtype=dtype)
    got = hbl.hbl_hadamard_f32(to_dev(x, dtype)).cpu().numpy().astype(np.float64)
    want = orc.hadamard(x)
    tol = 1e-5 * np.abs(want).max(axis=1, keepdims=True)
    assert np.all(np.abs(got - want) <= tol), float((np.abs(got - want) / tol).max())


def test_hadamard_unit_vectors_and_involution():
    K = 4096
    x = np.zeros((4, K), np.float32)
    x[0, 0] = 1; x[1, 1] = 1; x[2, K - 1] = 1; x[3, :] = 1
    got = hbl.hbl_hadamard_f32(to_dev(x, "f32")).cpu().numpy()
    idx = np.arange(K)
    s = 1 / 64.0
    assert np.array_equal(got[0], np.full(K, s, np.float32))
    assert np.array_equal(got[1], np.where(idx & 1, -s, s).astype(np.float32))
    par = np.array([bin(i).count("1") & 1 for i in idx])
    assert np.array_equal(got[2], np.where(par, -s, s).astype(np.float32))
    assert got[3, 0] == 64.0 and np.all(got[3, 1:] == 0)
    y = wl.rows("gauss", 1, 1, K, 0, 8, "f32")
    back = hbl.hbl_hadamard_f32(hbl.hbl_hadamard_f32(to_dev(y, "f32"))).cpu().numpy()
    assert np.allclose(back, y, atol=1e-5 * np.abs(y).max())


@pytest.mark.parametrize("K", [2048, 4096, 8192, 16384])
def test_hadamard_bf16_backward_matches_oracle(K):
    """The backward pass of the transform (the equation after Eq. 7 in the training section): the same
    orthonormal product applied to the gradient, bf16 in and out.  The oracle's transform in fp64 is the
    reference; the kernel computes in fp32 and rounds once to bf16, so an output may differ from the exact
    value by half a bf16 ulp (2^-9 relative) plus the fp32 error of log2 K butterfly stages, bounded here
    by 2^-18 of the row's largest output."""
    T = 37 if K <= 8192 else 9
    g = wl.rows("gauss", 300 + K, 1, K, 0, T, "bf16")
    got = hbl.hbl_hadamard_bf16(to_dev(g, "bf16")).float().cpu().numpy().astype(np.float64)
    want = orc.hadamard(g)
    tol = 2.0 ** -8 * np.abs(want) + 2.0 ** -18 * np.abs(want).max(axis=1, keepdims=True)
    assert np.all(np.abs(got - want) <= tol), float((np.abs(got - want) / tol).max())


def test_hadamard_bf16_exact_cases_and_involution():
    K = 8192                                   # 1/sqrt(K) is not a power of two here: one rounding in the scale
    x = np.zeros((3, K), np.float32)
    x[0, 5] = 1; x[1, :] = 1; x[2, 0] = 3; x[2, 1] = -3
    got = hbl.hbl_hadamard_bf16(to_dev(x, "bf16")).float().cpu().numpy()
    s = np.float32(1.0 / np.sqrt(np.float64(K)))
    sb = torch.tensor([s]).bfloat16().float().item()
    idx = np.arange(K)
    par5 = np.array([bin(i & 5).count("1") & 1 for i in idx])
    assert np.array_equal(got[0], np.where(par5, -sb, sb).astype(np.float32))          # column 5 of H, up to sign
    assert got[1, 0] == torch.tensor([K * s]).bfloat16().float().item() and np.all(got[1, 1:] == 0)
    want2 = np.where(idx & 1, 6 * s, 0).astype(np.float32)                              # 3 e0 - 3 e1
    assert np.array_equal(got[2], torch.from_numpy(want2).bfloat16().float().numpy())
    # applied twice it is the identity, up to the two bf16 roundings
    y = wl.rows("gauss", 2, 1, K, 0, 8, "bf16")
    yd = to_dev(y, "bf16")
    back = hbl.hbl_hadamard_bf16(hbl.hbl_hadamard_bf16(yd)).float().cpu().numpy()
    assert np.all(np.abs(back - y) <= 2.0 ** -7 * np.abs(y).max())
    # and it agrees with the fp32 export of the forward kernel, rounded
    f32 = hbl.hbl_hadamard_f32(yd)
    assert torch.equal(hbl.hbl_hadamard_bf16(yd), f32.bfloat16())


@pytest.mark.parametrize("K", ALL_K)
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("had", [True, False])
@pytest.mark.parametrize("prec", [32, 64])
def test_quantize_act_matches_oracle(K, bits, had, prec):
    """prec = 32: the oracle takes the rounding decision in IEEE fp32, as the kernel does; prec = 64: in fp64
    from the exact statistic, i.e. Eq. 5-6 as written.  The same rule holds against both: a code may differ
    by one only where the pre-rounding value is within 1e-5 (relative to the boundary, absolute below 1) of it."""
    T = 67 if K <= 8192 else 11
    kind = "ffn_mid" if K >= 8192 else "attn_out"
    x = make_x(K, T, 7 * K + bits, kind)
    codes, scale, csum = hbl.hbl_quantize_act(to_dev(x, "bf16"), bits, had, EPS)
    xr = orc.hadamard(x) if had else x.astype(np.float64)
    q, v, s, st = orc.act_quant(xr, bits, EPS, prec)
    cg = codes.cpu().numpy()
    check_codes(cg, q, v)
    assert np.allclose(scale.cpu().numpy(), s, rtol=2e-6, atol=0)
    assert np.array_equal(csum.cpu().numpy(), cg.astype(np.int64).sum(1))
    lo, hi = (-128, 127) if bits == 8 else (-8, 7)
    assert cg.min() >= lo and cg.max() <= hi


@pytest.mark.parametrize("bits", [4, 8])
def test_quantize_act_without_transform_is_bit_exact(bits):
    """No transform: the statistic is exact in fp32, so both sides take identical decisions
    (INT8: max is exact; INT4: the fp32 sum order may differ by an ulp, hence the tolerance rule)."""
    K, T = 4096, 130
    x = wl.rows("gauss", 4, 1, K, 0, T, "bf16")
    codes, scale, _ = hbl.hbl_quantize_act(to_dev(x, "bf16"), bits, False, EPS)
    q, v, s, st = orc.act_quant(x.astype(np.float64), bits, EPS, 32)
    if bits == 8:
        assert np.array_equal(codes.cpu().numpy(), q)
        assert np.array_equal(scale.cpu().numpy(), s.astype(np.float32))
    else:
        check_codes(codes.cpu().numpy(), q, v)


@pytest.mark.parametrize("K,T", [(16384, 70), (32768, 65), (11008, 66), (384, 131), (128, 203), (2048, 1025)])
@pytest.mark.parametrize("bits", [4, 8])
def test_quantize_act_without_transform_wide_and_odd_widths(K, T, bits):
    """bf16 rows of more than 64 tokens without the transform go through the row quantizer: the widest rows,
    widths that are not powers of two, a width below one warp's share, ragged token counts."""
    x = wl.rows("attn_out" if K < 8192 else "ffn_mid", 40 + bits, 1, K, 0, T, "bf16")
    codes, scale, csum = hbl.hbl_quantize_act(to_dev(x, "bf16"), bits, False, EPS)
    assert hbl.hbl_check_status() == 0
    q, v, s, st = orc.act_quant(x.astype(np.float64), bits, EPS, 32)
    cg = codes.cpu().numpy()
    check_codes(cg, q, v)
    assert np.allclose(scale.cpu().numpy(), s, rtol=2e-6, atol=0)
    assert np.array_equal(csum.cpu().numpy(), cg.astype(np.int64).sum(1))
    if bits == 8:
        assert np.array_equal(cg, q)                      # the maximum is exact: identical decisions


def test_quantize_act_generic_width_and_fp32_input():
    K, T = 384, 19                       # not a power of two: plain BitLinear input only
    x = wl.rows("gauss", 9, 1, K, 0, T, "f32")
    for bits in (4, 8):
        codes, scale, csum = hbl.hbl_quantize_act(to_dev(x, "f32"), bits, False, EPS)
        q, v, s, st = orc.act_quant(x.astype(np.float64), bits, EPS, 32)
        check_codes(codes.cpu().numpy(), q, v)
        assert np.allclose(scale.cpu().numpy(), s, rtol=2e-6)
        assert np.array_equal(csum.cpu().numpy(), codes.cpu().numpy().astype(np.int64).sum(1))
    with pytest.raises(hbl.HblError):
        hbl.hbl_quantize_act(to_dev(x, "f32"), 4, True, EPS)


def test_degenerate_tokens():
    K = 2048
    x = np.zeros((3, K), np.float32)
    x[1, 5] = 3.0                         # a single spike: the transform spreads it evenly
    x[2, :] = -2.0                        # constant: the transform concentrates it in index 0
    for bits in (4, 8):
        codes, scale, csum = hbl.hbl_quantize_act(to_dev(x, "bf16"), bits, True, EPS)
        c = codes.cpu().numpy(); sc = scale.cpu().numpy()
        assert np.all(c[0] == 0) and sc[0] == 0.0
        q, v, s, st = orc.act_quant(orc.hadamard(x), bits, EPS, 32)
        check_codes(c, q, v)
        assert np.all(np.isfinite(sc))
    assert hbl.hbl_quantize_act(torch.empty((0, K), dtype=torch.bfloat16, device="cuda"), 4, True, EPS)[0].shape[0] == 0
