"""GPU parity of the SwishGLU product fused in front of W_down's transform vs the oracle.

As with the fused normalisation, the oracle forms SiLU(gate) * up in fp64 and rounds once to bf16, the
kernel in fp32 (fast exponential, relative error ~2^-22); next to a bf16 rounding boundary the two land on
neighbouring values, which moves every transformed output of the token by at most 2^-8 |x'| / sqrt(K).
The transformed values are held to |dx_r| <= 1e-4 max_k |x_r|.  For everything after the rounding, the
kernel's own roundings are recovered and checked one by one (parity_utils.reconcile_bf16_inputs) and the
oracle continues from them, so codes, scales and outputs meet the plain layer's bars."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS, check_codes, check_y, reconcile_bf16_inputs, to_dev

pytestmark = pytest.mark.gpu


def gate_up(K, T, seed):
    g = wl.rows("gauss", seed, 1, K, 0, T, "bf16") * np.float32(2.0)      # still bf16-exact
    u = wl.rows("gauss", seed, 2, K, 0, T, "bf16")
    u[:, ::257] *= np.float32(32.0)                                       # a few outlier channels, as W_down's input has
    return g, u


@pytest.mark.parametrize("K", [2048, 4096, 8192, 16384])
def test_glu_transform_matches_oracle(K):
    T = 37 if K <= 8192 else 9
    g, u = gate_up(K, T, 1100 + K)
    xg, _ = orc.swiglu_bf16(g, u)
    want = orc.hadamard(xg)
    got = hbl.hbl_glu_quantize_act(to_dev(g, "bf16"), to_dev(u, "bf16"), 4, EPS, export_xr=True).cpu().numpy().astype(np.float64)
    tol = 1e-4 * np.abs(want).max(axis=1, keepdims=True)
    assert np.all(np.abs(got - want) <= tol), float((np.abs(got - want) / tol).max())


def test_glu_special_cases():
    K = 4096
    # gate = 0 gives a zero token whatever `up` is; very negative gates give (minus) zero, not NaN
    z = torch.zeros((2, K), dtype=torch.bfloat16, device="cuda")
    u = torch.randn((2, K), device="cuda").bfloat16()
    codes, scale, csum = hbl.hbl_glu_quantize_act(z, u, 4, EPS)
    assert not codes.any() and not csum.any()
    neg = torch.full((2, K), -200.0, dtype=torch.bfloat16, device="cuda")
    xr = hbl.hbl_glu_quantize_act(neg, u, 4, EPS, export_xr=True)
    assert torch.isfinite(xr).all() and not xr.any()
    # large positive gates pass `up` through: SiLU(z) = z there, so x' = z * up exactly when the product is bf16-exact
    big = torch.full((1, K), 64.0, dtype=torch.bfloat16, device="cuda")
    u1 = torch.zeros((1, K), dtype=torch.bfloat16, device="cuda"); u1[0, 3] = 0.5
    xr = hbl.hbl_glu_quantize_act(big, u1, 4, EPS, export_xr=True).cpu().numpy()
    want = orc.hadamard((big.float() * u1.float()).cpu().numpy())
    assert np.allclose(xr, want, rtol=0, atol=1e-5 * np.abs(want).max())
    assert hbl.hbl_check_status() == 0


@pytest.mark.parametrize("bits", [4, 8])
def test_glu_quantize_matches_oracle(bits):
    K, T = 8192, 41
    g, u = gate_up(K, T, 1300 + bits)
    gd, ud = to_dev(g, "bf16"), to_dev(u, "bf16")
    xg, pre = orc.swiglu_bf16(g, u)
    xk, n_moved = reconcile_bf16_inputs(hbl.hbl_glu_quantize_act(gd, ud, bits, EPS, export_xr=True), xg, pre)
    assert n_moved <= 1e-3 * xg.size
    q, v, s, st = orc.act_quant(orc.hadamard(xk), bits, EPS, 32)
    codes, scale, csum = hbl.hbl_glu_quantize_act(gd, ud, bits, EPS)
    cg = codes.cpu().numpy()
    # the gating product has channels 30 times the rest (max |x_r| / beta, which scales the fp32 butterflies'
    # error into code units, is a few times larger than on the plain layer's inputs), and elements too small to
    # recover from the export may have been rounded the other way unnoticed
    check_codes(cg, q, v, near=4e-5)
    assert np.allclose(scale.cpu().numpy(), s, rtol=5e-5, atol=0)      # fp32 butterflies vs fp64 on heavy-tailed rows
    assert np.array_equal(csum.cpu().numpy(), cg.astype(np.int64).sum(1))


@pytest.mark.parametrize("T", [5, 16, 300])
def test_forward_glu_matches_oracle(T):
    K, N = 4096, 528
    g, u = gate_up(K, T, 1500 + T)
    W = wl.rows("latent", 1500 + T, 3, K, 0, N, "f32")
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    y = hbl.hbl_forward_glu(to_dev(g, "bf16"), to_dev(u, "bf16"), packed, alpha, N, 4, EPS)
    assert hbl.hbl_check_status() == 0
    gd, ud = to_dev(g, "bf16"), to_dev(u, "bf16")
    xg, pre = orc.swiglu_bf16(g, u)
    xk, n_moved = reconcile_bf16_inputs(hbl.hbl_glu_quantize_act(gd, ud, 4, EPS, export_xr=True), xg, pre)
    assert n_moved <= 1e-3 * xg.size
    wt, al = orc.weight_quant(W, EPS, 32)
    q, v, s, st = orc.act_quant(orc.hadamard(xk), 4, EPS, 32)
    _, y64 = orc.rescale(orc.gemm(q, wt), s, al)
    check_y(y, y64)
    # the plain layer on the product formed outside (with the kernel's roundings) gives the same values
    # (up to roundings of elements too small to recover from the export, which can move a code or two)
    y2 = hbl.hbl_forward(to_dev(xk, "bf16"), packed, alpha, N, 4, True, EPS).float()
    rms = y2.pow(2).mean(1, keepdim=True).sqrt()
    assert torch.all((y.float() - y2).abs() <= 1e-2 * torch.maximum(y2.abs(), rms))
    assert (y.float() != y2).float().mean() <= 1e-2


@pytest.mark.parametrize("T", [7, 300])
def test_block_chains_the_feed_forward(T):
    """hbl_block_forward without a down input: the down projection takes SiLU(ygate) * yup from the outputs the
    same call has just written.  It must give what hbl_forward_glu gives on those two outputs, on either path,
    and leave the other six outputs as the unchained call does."""
    H, F = 512, 2048
    seed = 41
    ins = {"attn_in": wl.rows("gauss", seed, 10, H, 0, T, "bf16"), "o_in": wl.rows("attn_out", seed, 11, H, 0, T, "bf16"),
           "ffn_in": wl.rows("gauss", seed, 12, H, 0, T, "bf16")}
    shapes = {"q": (H, H), "k": (H, H), "v": (H, H), "o": (H, H), "up": (F, H), "gate": (F, H), "down": (H, F)}
    packed, alphas = {}, []
    for i, (n, sh) in enumerate(shapes.items()):
        p, a = hbl.hbl_quantize_weights(torch.from_numpy(wl.rows("latent", seed, 20 + i, sh[1], 0, sh[0], "f32")).cuda(), EPS)
        packed[n] = p
        alphas.append(a)
    alpha7 = torch.cat(alphas)
    dev = {k: to_dev(v, "bf16") for k, v in ins.items()}
    for path in (hbl.PATH_AUTO, hbl.PATH_TENSOR):
        outs = hbl.hbl_block_forward(dev, packed, alpha7, H, F, 4, EPS, path=path)
        assert hbl.hbl_check_status() == 0
        want_down = hbl.hbl_forward_glu(outs["gate"], outs["up"], packed["down"], alphas[6], H, 4, EPS, path=path)
        assert torch.equal(outs["down"], want_down)
        full = dict(dev, down_in=torch.zeros((T, F), dtype=torch.bfloat16, device="cuda"))
        ref = hbl.hbl_block_forward(full, packed, alpha7, H, F, 4, EPS, path=path)
        for n in ("q", "k", "v", "o", "up", "gate"):
            assert torch.equal(outs[n], ref[n])
