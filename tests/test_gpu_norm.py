"""GPU parity of the normalisation fused in front of the transform ("LN" of Eq. 7) vs the oracle.

The oracle normalises in fp64 and rounds once to bf16; the kernel normalises in fp32 and rounds once to
bf16.  Where the exact value lies next to a bf16 rounding boundary the two may land on neighbouring bf16
values; such an element moves every transformed output of its token by at most 2^-8 |x'| / sqrt(K).  The
tests bound how often that happens through what it does downstream:
  * transformed values: |dx_r| <= 1e-4 max_k |x_r| (1e-5 for the fp32 butterflies plus the moved inputs);
  * everything after the rounding: the kernel's own roundings are recovered and checked one by one
    (parity_utils.reconcile_bf16_inputs) and the oracle continues from them, so codes, scales and outputs
    meet the plain layer's bars."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS, check_codes, check_y, reconcile_bf16_inputs, to_dev

pytestmark = pytest.mark.gpu
NORM_EPS = 1e-5


def gain_vector(K, seed):
    rng = np.random.default_rng(seed)
    return rng.uniform(0.25, 2.0, K).astype(np.float32)


@pytest.mark.parametrize("gain_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("K", [2048, 4096, 8192, 16384])
def test_norm_transform_matches_oracle(K, gain_dtype):
    T = 37 if K <= 8192 else 9
    x = wl.rows("ffn_mid" if K >= 8192 else "attn_out", 500 + K, 1, K, 0, T, "bf16")
    g = gain_vector(K, K)
    gd = torch.from_numpy(g).cuda()
    if gain_dtype == "bf16":                                  # the oracle sees the gain the kernel sees
        gd = gd.bfloat16()
        g = gd.float().cpu().numpy()
    xn, _ = orc.rmsnorm_bf16(x, g, NORM_EPS)
    want = orc.hadamard(xn)
    got = hbl.hbl_norm_quantize_act(to_dev(x, "bf16"), gd, NORM_EPS, 4, EPS, export_xr=True)
    got = got.cpu().numpy().astype(np.float64)
    tol = 1e-4 * np.abs(want).max(axis=1, keepdims=True)
    assert np.all(np.abs(got - want) <= tol), float((np.abs(got - want) / tol).max())


def test_norm_special_cases():
    K = 4096
    g = gain_vector(K, 3)
    gd = torch.from_numpy(g).cuda()
    # a constant token normalises to the gain vector (exactly, for a gain that is bf16-exact)
    gb = torch.from_numpy(g).bfloat16().float()
    x = np.full((2, K), 3.0, np.float32); x[1] = -0.5
    xr = hbl.hbl_norm_quantize_act(to_dev(x, "bf16"), gb.cuda(), 0.0, 4, EPS, export_xr=True).cpu().numpy()
    want = orc.hadamard(np.stack([gb.numpy(), -gb.numpy()]))
    assert np.all(np.abs(xr - want) <= 1e-5 * np.abs(want).max(axis=1, keepdims=True))
    # scaling a token by a power of two changes nothing when norm_eps is zero
    y = wl.rows("gauss", 9, 1, K, 0, 6, "bf16")
    a = hbl.hbl_norm_quantize_act(to_dev(y, "bf16"), gd, 0.0, 4, EPS)
    b = hbl.hbl_norm_quantize_act(to_dev(4 * y, "bf16"), gd, 0.0, 4, EPS)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    # an all-zero token gives zero codes
    z = torch.zeros((3, K), dtype=torch.bfloat16, device="cuda")
    codes, scale, csum = hbl.hbl_norm_quantize_act(z, gd, NORM_EPS, 8, EPS)
    assert not codes.any() and not csum.any() and hbl.hbl_check_status() == 0


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("K", [2048, 8192])
def test_norm_quantize_matches_oracle(K, bits):
    T = 41
    x = wl.rows("attn_out", 700 + K + bits, 1, K, 0, T, "bf16")
    g = gain_vector(K, K + 1)
    xd, gd = to_dev(x, "bf16"), torch.from_numpy(g).cuda()
    xn, pre = orc.rmsnorm_bf16(x, g, NORM_EPS)
    xk, n_moved = reconcile_bf16_inputs(hbl.hbl_norm_quantize_act(xd, gd, NORM_EPS, bits, EPS, export_xr=True), xn, pre)
    assert n_moved <= 1e-3 * xn.size
    q, v, s, st = orc.act_quant(orc.hadamard(xk), bits, EPS, 32)
    codes, scale, csum = hbl.hbl_norm_quantize_act(xd, gd, NORM_EPS, bits, EPS)
    cg = codes.cpu().numpy()
    # elements too small to recover from the export may have been rounded the other way unnoticed: each moves
    # the pre-rounding values by ~1e-5, on top of the fp32 butterflies' own error
    check_codes(cg, q, v, near=4e-5)
    assert np.allclose(scale.cpu().numpy(), s, rtol=5e-5, atol=0)      # fp32 butterflies vs fp64 on heavy-tailed rows
    assert np.array_equal(csum.cpu().numpy(), cg.astype(np.int64).sum(1))


@pytest.mark.parametrize("T", [5, 16, 300])
def test_forward_norm_matches_oracle(T):
    K, N = 2048, 784
    x = wl.rows("attn_out", 900 + T, 1, K, 0, T, "bf16")
    W = wl.rows("latent", 900 + T, 2, K, 0, N, "f32")
    g = gain_vector(K, T)
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    y = hbl.hbl_forward_norm(to_dev(x, "bf16"), torch.from_numpy(g).cuda(), NORM_EPS, packed, alpha, N, 4, EPS)
    assert hbl.hbl_check_status() == 0
    xd, gd = to_dev(x, "bf16"), torch.from_numpy(g).cuda()
    if T == 16:                                               # one of the cases with a bf16 gain
        gd = gd.bfloat16()
        g = gd.float().cpu().numpy()
        y = hbl.hbl_forward_norm(xd, gd, NORM_EPS, packed, alpha, N, 4, EPS)
    xn, pre = orc.rmsnorm_bf16(x, g, NORM_EPS)
    xk, n_moved = reconcile_bf16_inputs(hbl.hbl_norm_quantize_act(xd, gd, NORM_EPS, 4, EPS, export_xr=True), xn, pre)
    assert n_moved <= 1e-3 * xn.size
    wt, al = orc.weight_quant(W, EPS, 32)
    q, v, s, st = orc.act_quant(orc.hadamard(xk), 4, EPS, 32)
    _, y64 = orc.rescale(orc.gemm(q, wt), s, al)
    check_y(y, y64)
    # the plain layer applied to the normalised activations (with the kernel's roundings) gives the same values
    # (up to roundings of elements too small to recover from the export, which can move a code or two)
    y2 = hbl.hbl_forward(to_dev(xk, "bf16"), packed, alpha, N, 4, True, EPS).float()
    rms = y2.pow(2).mean(1, keepdim=True).sqrt()
    assert torch.all((y.float() - y2).abs() <= 1e-2 * torch.maximum(y2.abs(), rms))
    assert (y.float() != y2).float().mean() <= 1e-2
