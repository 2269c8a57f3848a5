"""Pins for the CPU oracle: closed forms, invariants, hand-worked values, library
routines on special cases and brute force on tiny inputs.  None of these retype
the oracle's own butterfly / quantizer code: each checks it against something
the mathematics fixes independently."""
import json
import math
import os

import numpy as np
import pytest

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import workloads as wl

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")))
EPS = 1e-5
PRECS = (32, 64)


def Phi(z):
    return 0.5 * (1.0 + math.erf(z / math.sqrt(2.0)))


# ------------------------------------------------------------------ Hadamard
def popcount_matrix(n):
    """Entry closed form of the Sylvester matrix: H[i,j] = (-1)^popcount(i&j)."""
    H = np.empty((n, n))
    for i in range(n):
        for j in range(n):
            H[i, j] = -1.0 if bin(i & j).count("1") & 1 else 1.0
    return H


@pytest.mark.parametrize("n", [1, 2, 4, 8, 16, 32, 64])
def test_hadamard_matches_popcount_closed_form(n):
    rng = np.random.default_rng(n)
    x = rng.standard_normal((5, n)).astype(np.float32)
    want = x.astype(np.float64) @ popcount_matrix(n).T / math.sqrt(n)
    got = orc.hadamard(x)
    assert np.allclose(got, want, rtol=0, atol=1e-13 * n)


@pytest.mark.parametrize("n", [2, 16, 256])
def test_hadamard_matches_kronecker_and_scipy(n):
    from scipy.linalg import hadamard as scipy_hadamard
    H2 = np.array([[1.0, 1.0], [1.0, -1.0]])
    H = np.array([[1.0]])
    while H.shape[0] < n:
        H = np.kron(H2, H)          # the recursion of Eq. 4 without the 1/sqrt(2)
    assert np.array_equal(H, scipy_hadamard(n).astype(np.float64))
    got = orc.hadamard(np.eye(n, dtype=np.float32)) * math.sqrt(n)   # rows = H e_i
    assert np.allclose(got, H, atol=1e-12)
    assert np.allclose(got @ got.T, n * np.eye(n), atol=1e-9)        # H H^T = n I


@pytest.mark.parametrize("case", GOLD["hadamard"], ids=lambda c: c["cite"])
def test_hadamard_hand_values(case):
    x = np.array([case["x"]], dtype=np.float32)
    got = orc.hadamard(x)[0] * math.sqrt(len(case["x"]))
    assert np.allclose(got, case["xr_times_sqrt_n"], atol=1e-12)


@pytest.mark.parametrize("n", [8, 512, 4096, 16384])
def test_hadamard_invariants(n):
    rng = np.random.default_rng(n + 1)
    x = rng.standard_normal((3, n)).astype(np.float32)
    y = orc.hadamard(x)
    # Parseval (orthonormal)
    assert np.allclose((y ** 2).sum(1), (x.astype(np.float64) ** 2).sum(1), rtol=1e-12)
    # involution: the transform applied twice returns the input (inputs kept fp32-exact)
    y32 = y.astype(np.float32)
    back = orc.hadamard(y32)
    assert np.allclose(back, x, atol=1e-5 * np.abs(x).max())
    # e_0 -> 1/sqrt(n); all-ones -> sqrt(n) e_0
    e0 = np.zeros((1, n), np.float32); e0[0, 0] = 1
    assert np.allclose(orc.hadamard(e0), 1 / math.sqrt(n), atol=1e-15)
    ones = orc.hadamard(np.ones((1, n), np.float32))[0]
    assert abs(ones[0] - math.sqrt(n)) < 1e-10 and np.abs(ones[1:]).max() < 1e-10
    # e_j -> column j of H: sign pattern (-1)^popcount(i&j), natural order
    j = n // 2 + 1 if n > 2 else 1
    ej = np.zeros((1, n), np.float32); ej[0, j] = 1
    col = orc.hadamard(ej)[0] * math.sqrt(n)
    idx = np.arange(n)
    pc = np.array([bin(int(i) & j).count("1") & 1 for i in idx])
    assert np.array_equal(col, np.where(pc == 1, -1.0, 1.0))
    # linearity (exact inputs)
    a = np.float32(0.5); b = np.float32(-2.0)
    lin = orc.hadamard((a * x[0:1] + b * x[1:2]).astype(np.float32))
    # (a*x0+b*x1 is rounded to fp32 before the call; compare against the rounded input's transform)
    assert np.allclose(lin, a * y[0:1] + b * y[1:2], atol=1e-5)


def test_hadamard_rejects_non_power_of_two():
    with pytest.raises(RuntimeError):
        orc.hadamard(np.zeros((1, 12), np.float32))


# ------------------------------------------------------------------ quantizers
@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("case", GOLD["int4"], ids=lambda c: c["cite"])
def test_int4_hand_values(case, prec):
    x = np.array([case["x"]], dtype=np.float64)
    q, v, s, st = orc.act_quant(x, 4, EPS, prec)
    assert q[0].tolist() == case["codes"]
    assert abs(st[0] - case["beta"]) < 1e-6
    assert abs(s[0] - case["s"]) < 1e-6
    assert np.all(np.isfinite(v))


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("case", GOLD["int8"], ids=lambda c: c["cite"])
def test_int8_hand_values(case, prec):
    x = np.array([case["x"]], dtype=np.float64)
    q, v, s, st = orc.act_quant(x, 8, case.get("eps", EPS), prec)
    assert q[0].tolist() == case["codes"]
    assert abs(st[0] - case["gamma"]) < 1e-6
    assert abs(s[0] - case["s"]) < 1e-6


@pytest.mark.parametrize("prec", PRECS)
def test_int4_code_distribution_on_gaussian(prec):
    """For x ~ N(0,1), beta -> sqrt(2/pi); the code histogram follows from Phi."""
    K, T = 16384, 64
    rng = np.random.default_rng(7)
    x = rng.standard_normal((T, K))
    q, v, s, st = orc.act_quant(x, 4, EPS, prec)
    beta = math.sqrt(2 / math.pi)
    assert abs(st.mean() - beta) < 2e-3
    c = math.sqrt(7) / beta                      # v = c * x
    def p_code(k):
        lo = -math.inf if k == -8 else (k - 0.5) / c
        hi = math.inf if k == 7 else (k + 0.5) / c
        return Phi(hi) - Phi(lo)
    n = q.size
    for k in range(-8, 8):
        want = p_code(k)
        got = np.count_nonzero(q == k) / n
        assert abs(got - want) < 5 * math.sqrt(want * (1 - want) / n) + 2e-4, (k, got, want)
    assert abs(p_code(7) - 0.0250) < 2e-4 and abs(p_code(-8) - 0.0119) < 2e-4
    assert q.min() == -8 and q.max() == 7


@pytest.mark.parametrize("prec", PRECS)
def test_int8_never_reaches_minus_128_and_hits_127(prec):
    rng = np.random.default_rng(8)
    x = rng.standard_normal((32, 1024)) * 3.0
    q, v, s, st = orc.act_quant(x, 8, EPS, prec)
    assert q.min() >= -127 and q.max() <= 127
    # the absmax entry of every token maps to +-127
    am = np.abs(x).argmax(1)
    assert np.all(np.abs(q[np.arange(32), am].astype(int)) == 127)
    assert np.allclose(st, np.abs(x).max(1), rtol=1e-6)
    assert np.allclose(s, st / 127.0, rtol=1e-12)


@pytest.mark.parametrize("bits", [4, 8])
def test_quantizer_dequant_error_bound(bits):
    """Away from clipping, |s*q - x*stat/(stat+eps)| <= s/2 (round to nearest)."""
    rng = np.random.default_rng(9)
    x = rng.standard_normal((8, 2048))
    q, v, s, st = orc.act_quant(x, bits, EPS, 64)
    hi = 127 if bits == 8 else 7
    lo = -128 if bits == 8 else -8
    inside = (v > lo - 0.5) & (v < hi + 0.5)
    err = np.abs(s[:, None] * q - x * (st / (st + EPS))[:, None])
    assert np.all(err[inside] <= 0.5 * np.broadcast_to(s[:, None], err.shape)[inside] * (1 + 1e-9))
    assert np.all(q[v >= hi + 0.5] == hi) and np.all(q[v <= lo - 0.5] == lo)


def test_bits_must_be_4_or_8():
    with pytest.raises(RuntimeError):
        orc.act_quant(np.zeros((1, 4)), 5, EPS, 64)


# ------------------------------------------------------------------ ternary weights
@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("case", GOLD["ternary"], ids=lambda c: c["cite"])
def test_ternary_hand_values(case, prec):
    wt, alpha = orc.weight_quant(np.array(case["W"], np.float32), EPS, prec)
    assert abs(float(alpha) - case["alpha"]) < 1e-7
    assert wt.tolist() == case["wt"]


@pytest.mark.parametrize("prec", PRECS)
def test_ternary_statistics_on_gaussian_latents(prec):
    sigma = 0.02
    W = wl.rows("latent", 123, 1, 2048, 0, 1024)
    wt, alpha = orc.weight_quant(W, EPS, prec)
    assert abs(float(alpha) / sigma - math.sqrt(2 / math.pi)) < 2e-3
    # w = 0 iff |W| < (alpha+eps)/2  (up to the tie)
    z = 0.5 * (float(alpha) + EPS) / sigma
    p0 = 2 * Phi(z) - 1
    n = wt.size
    assert abs(np.count_nonzero(wt == 0) / n - p0) < 5 * math.sqrt(p0 * (1 - p0) / n)
    assert abs(p0 - 0.310) < 2e-3
    assert abs(np.count_nonzero(wt == 1) / n - (1 - p0) / 2) < 3e-3
    assert set(np.unique(wt).tolist()) == {-1, 0, 1}
    # independent restatement of the decision on a sample, in exact rational-free form:
    # |W| > (alpha+eps)/2 <=> |w| = 1 and sign(w) = sign(W)
    thr = 0.5 * (np.float64(alpha) + EPS)
    far = np.abs(np.abs(W.astype(np.float64)) - thr) > 1e-7
    assert np.array_equal(wt[far], (np.sign(W) * (np.abs(W.astype(np.float64)) > thr))[far].astype(np.int8))


def test_ternary_alpha_is_fp64_mean_rounded_once():
    W = wl.rows("latent", 5, 9, 512, 0, 512)
    _, alpha = orc.weight_quant(W, EPS, 64)
    want = np.float32(math.fsum(np.abs(W.astype(np.float64)).ravel().tolist()) / W.size)
    assert alpha == want


# ------------------------------------------------------------------ contraction and rescale
@pytest.mark.parametrize("k", [1, 2, 77, 4095, 0x3FFFFF])
def test_ternary_decision_at_the_rounding_threshold(k):
    """Eq. 1-2 with round-half-to-even: W_t = sign(w) exactly where |w| / (alpha + eps) rounds above 1/2, which
    in exact arithmetic is |w| > (alpha + eps) / 2, a tie going to 0.  The tensor fixes alpha exactly (every
    group of four magnitudes adds up to 4 a), makes alpha + eps = 1 + k 2^-23, and puts the first entry of each
    group on the threshold or a few fp32 steps beside it.  Entries of magnitude ~1.6 d check the clip."""
    N, K = 16, 128
    eps = 2.0 ** -17
    d = 1.0 + k * 2.0 ** -23
    a, h = d - eps, d / 2
    mag = np.full(N * K, a)
    x = h + (np.arange(N * K // 4) % 9 - 4) * 2.0 ** -24
    mag[0::4] = x
    mag[1::4] = 0.75 - x
    mag[2::4] = mag[3::4] = (4 * a - 0.75) / 2
    assert np.array_equal(mag.astype(np.float32).astype(np.float64), mag)       # every entry is an fp32 value
    sign = np.where(np.arange(N * K) % 3 == 0, -1.0, 1.0)
    W = (mag * sign).astype(np.float32).reshape(N, K)
    for prec in (32, 64):
        wt, al = orc.weight_quant(W, eps, prec)
        assert al == np.float32(a)
        want = np.where(mag > h, sign, 0.0).astype(np.int8).reshape(N, K)
        assert np.array_equal(wt, want)
        assert np.count_nonzero(wt.reshape(-1)[0::4] == 0) > 100 and np.count_nonzero(wt.reshape(-1)[0::4]) > 100


def test_gemm_matches_fp64_matmul_and_special_cases():
    rng = np.random.default_rng(11)
    q = rng.integers(-128, 128, size=(7, 96), dtype=np.int8)
    wt = rng.integers(-1, 2, size=(13, 96), dtype=np.int8)
    acc = orc.gemm(q, wt)
    assert np.array_equal(acc, (q.astype(np.float64) @ wt.astype(np.float64).T).astype(np.int64))
    assert np.array_equal(orc.gemm(q, np.ones((3, 96), np.int8)), np.repeat(q.astype(np.int64).sum(1)[:, None], 3, 1))
    onehot = np.zeros((96, 96), np.int8); onehot[np.arange(96), np.arange(96)[::-1]] = -1
    assert np.array_equal(orc.gemm(q, onehot), -q[:, ::-1].astype(np.int32))
    # extreme magnitudes: K=16384 of (-128)*(-1) stays inside int32
    K = 16384
    assert orc.gemm(np.full((1, K), -128, np.int8), np.full((1, K), -1, np.int8))[0, 0] == 128 * K


def test_rescale_rounds_once_to_bf16():
    import torch
    acc = np.array([[1, 3, -5, 257, 129, 131, 0, 7]], dtype=np.int32)
    yb, y64 = orc.rescale(acc, np.array([1.0]), 1.0)
    # 257 = 1.00000001b*2^8 lies exactly between 256 and 258 -> even significand (256);
    # 129 (between 128 and 130 in bf16? no: 129 = 10000001b is exact, 8 bits) stays.
    want = torch.tensor(acc[0].astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(yb[0], want)
    assert orc.bf16_bits_to_f32(yb)[0].tolist() == [1.0, 3.0, -5.0, 256.0, 129.0, 131.0, 0.0, 7.0]
    # ties at the 9th significand bit go to even: 1+2^-8 -> 1, 1+3*2^-8 -> 1+2^-6
    yb, _ = orc.rescale(np.array([[1 << 20]], np.int32), np.array([(1 + 2.0 ** -8) / (1 << 20)]), 1.0)
    assert orc.bf16_bits_to_f32(yb)[0, 0] == 1.0
    yb, _ = orc.rescale(np.array([[1 << 20]], np.int32), np.array([(1 + 3 * 2.0 ** -8) / (1 << 20)]), 1.0)
    assert orc.bf16_bits_to_f32(yb)[0, 0] == 1.0 + 2.0 ** -6
    # a value just above a tie must round up even though (float) would land on the tie first
    v = 1 + 2.0 ** -8 + 2.0 ** -40
    yb, _ = orc.rescale(np.array([[1]], np.int32), np.array([v]), 1.0)
    assert orc.bf16_bits_to_f32(yb)[0, 0] == 1.0 + 2.0 ** -7
    # random values against torch's fp32->bf16 on fp32-exact products
    rng = np.random.default_rng(3)
    acc = rng.integers(-100000, 100000, size=(4, 64)).astype(np.int32)
    yb, y64 = orc.rescale(acc, np.array([0.5, 0.25, 2.0, 1.0]), 0.125)
    want = torch.tensor(y64.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(yb, want)


def test_rescale_below_the_smallest_normal_bf16():
    """Outputs below 2^-126 take the subnormal branch of the rounding: bf16 subnormals are the multiples of
    2^-133 (7 fraction bits under an exponent of -126), ties go to the even multiple, and the top of the range
    carries into the smallest normal.  Each expected value is written out from that definition; the last check
    holds the whole branch against the fp32 -> bf16 conversion of a library on fp32-exact inputs."""
    import torch
    u = 2.0 ** -133                                        # spacing of bf16 subnormals
    cases = [
        (1, 1.0 * u, 0x0001), (1, 5.0 * u, 0x0005), (-1, 5.0 * u, 0x8005), (3, 9.0 * u, 27),
        (1, 0.5 * u, 0x0000),                              # tie between 0 and u: even (0)
        (1, 1.5 * u, 0x0002),                              # tie between u and 2u: even (2u)
        (1, 2.5 * u, 0x0002),                              # tie between 2u and 3u: even (2u)
        (1, 2.5 * u * (1 + 2.0 ** -30), 0x0003),           # just above that tie
        (1, 0.49 * u, 0x0000), (-1, 0.49 * u, 0x8000),     # underflow keeps the sign
        (1, 127.0 * u, 0x007F),                            # the largest subnormal
        (1, 127.5 * u, 0x0080),                            # tie at the top: even = 128 u = 2^-126, the smallest normal
        (1, 127.4 * u, 0x007F),
        (1, 2.0 ** -126, 0x0080), (1, 2.0 ** -127, 0x0040),
    ]
    for a, s, bits in cases:
        yb, y64 = orc.rescale(np.array([[a]], np.int32), np.array([s]), 1.0)
        assert yb[0, 0] == bits, (a, s, hex(int(yb[0, 0])), hex(bits))
        assert y64[0, 0] == a * s
    rng = np.random.default_rng(11)
    mant = rng.integers(1, 1 << 20, size=(1, 256)).astype(np.int32)            # fp32-exact subnormal products
    yb, y64 = orc.rescale(mant, np.array([2.0 ** -146]), 1.0)                  # values in (0, 2^-126)
    assert np.all(y64 < 2.0 ** -126) and np.array_equal(y64.astype(np.float32).astype(np.float64), y64)
    want = torch.tensor(y64.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(yb, want)


@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("case", GOLD["layer"], ids=lambda c: c["cite"])
def test_layer_hand_values(case, prec):
    W = np.array(GOLD["ternary"][0]["W"], np.float32)
    wt, alpha = orc.weight_quant(W, EPS, prec)
    x = np.array([case["x"]], np.float32)
    out = orc.forward(x, wt, alpha, case["bits"], bool(case["use_hadamard"]), EPS, prec, want_stages=True)
    assert out["codes"][0].tolist() == case["codes"]
    assert out["acc"][0].tolist() == case["acc"]
    assert np.allclose(out["y64"][0], case["y"], atol=2e-5)
    import torch
    want_bf16 = torch.tensor(case["y"], dtype=torch.float64).to(torch.float32).to(torch.bfloat16).float().numpy()
    assert np.array_equal(orc.bf16_bits_to_f32(out["y_bits"])[0], want_bf16)


def test_forward_equals_its_stages_and_dense_definition():
    """Eq. 7 written densely: y = (alpha*W_t) @ (s*q), with x_r from the dense popcount matrix."""
    n, N, T = 64, 24, 5
    rng = np.random.default_rng(21)
    x = rng.standard_normal((T, n)).astype(np.float32)
    x[:, 3] *= 40
    W = (rng.standard_normal((N, n)) * 0.02).astype(np.float32)
    wt, alpha = orc.weight_quant(W, EPS, 64)
    out = orc.forward(x, wt, alpha, 4, True, EPS, 64, want_stages=True)
    xr = x.astype(np.float64) @ popcount_matrix(n) / math.sqrt(n)
    beta = np.abs(xr).mean(1, keepdims=True)
    q = np.clip(np.rint(xr * math.sqrt(7) / (beta + EPS)), -8, 7)
    y = (q * beta / math.sqrt(7)) @ (float(alpha) * wt.astype(np.float64)).T
    assert np.array_equal(out["codes"], q.astype(np.int8))
    assert np.allclose(out["y64"], y, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ properties of the layer
def test_rotation_identity_without_quantization():
    """W x = (W H)(H x): the transform is orthogonal, so rotating both sides changes nothing."""
    n = 256
    rng = np.random.default_rng(5)
    x = rng.standard_normal((4, n)).astype(np.float32)
    W = rng.standard_normal((16, n)).astype(np.float32)
    lhs = x.astype(np.float64) @ W.astype(np.float64).T
    rhs = orc.hadamard(x) @ orc.hadamard(W).T
    assert np.allclose(lhs, rhs, atol=1e-9)


@pytest.mark.parametrize("bits", [4, 8])
def test_token_scaling_and_permutation(bits):
    wlc = wl.CONFIG1
    x = wlc.x(0, 8)
    wt, alpha = orc.weight_quant(wlc.w_latent(), EPS, 64)
    base = orc.forward(x, wt, alpha, bits, True, EPS, 64, want_stages=True)
    sc = orc.forward((x * np.float32(4.0)), wt, alpha, bits, True, EPS, 64, want_stages=True)
    assert np.array_equal(base["codes"], sc["codes"])          # eps shift is far below any boundary here
    assert np.allclose(sc["y64"], 4.0 * base["y64"], rtol=1e-12)
    perm = np.array([3, 1, 7, 0, 2, 6, 5, 4])
    pm = orc.forward(x[perm], wt, alpha, bits, True, EPS, 64)
    assert np.array_equal(pm["y_bits"], base["y_bits"][perm])


def test_hadamard_removes_outlier_channels_on_the_workloads():
    """Section 2.1's qualitative claim on the synthetic stand-ins: after the transform the
    per-token max/mean ratio collapses and INT4 round-trip error drops."""
    for cfg in (wl.CONFIG1, wl.CONFIG2, wl.CONFIG3):
        x = cfg.x(0, 16)
        xr = orc.hadamard(x)
        r_before = (np.abs(x).max(1) / np.abs(x).mean(1)).mean()
        r_after = (np.abs(xr).max(1) / np.abs(xr).mean(1)).mean()
        assert r_after < 0.25 * r_before, (cfg.name, r_before, r_after)
        assert r_after < 8.0                      # Gaussian-like: max/mean ~ 4-6 for these K
        def rel_mse(v):
            q, _, s, _ = orc.act_quant(v, 4, EPS, 64)
            return (((q * s[:, None]) - v) ** 2).sum() / (v ** 2).sum()
        assert rel_mse(xr) < 0.5 * rel_mse(x.astype(np.float64)), cfg.name


def test_layer_tracks_the_unquantized_product_with_int8():
    cfg = wl.CONFIG1
    x = cfg.x(0, 16)
    wt, alpha = orc.weight_quant(cfg.w_latent(), EPS, 64)
    out = orc.forward(x, wt, alpha, 8, True, EPS, 64)
    ref = orc.hadamard(x) @ (float(alpha) * wt.astype(np.float64)).T
    rel = np.linalg.norm(out["y64"] - ref) / np.linalg.norm(ref)
    assert rel < 0.02


# ------------------------------------------------------------------ generators
def test_workload_rows_are_reproducible_and_blockwise():
    a = wl.rows("attn_out", 2, 1, 2048, 0, 200, "bf16")
    b = wl.rows("attn_out", 2, 1, 2048, 130, 50, "bf16")
    assert np.array_equal(a[130:180], b)
    assert np.array_equal(wl.round_to_bf16(a)[0], a)
    ch = wl.outlier_channels(2, 1, 2048, 0.005)
    assert len(ch) == 10
    col_rms = np.sqrt((a ** 2).mean(0))
    assert col_rms[ch].min() > 10 * np.median(col_rms)
    assert wl.CONFIG1.x(0, 64).shape == (64, 512)
    assert len(wl.outlier_channels(0, 1, 512, 0.01)) == 5
    assert len(wl.outlier_channels(3, 1, 8192, 0.002)) == 16
    w = wl.CONFIG2.w_latent(0, 64)
    assert abs(w.std() - 0.02) < 5e-4


# ------------------------------------------------------------------ normalisation in front of the transform
def test_rmsnorm_hand_values_and_closed_forms():
    # 3-4-0-0: mean square 25/4, rms 2.5 -> 1.2, 1.6, 0, 0; in bf16 (8 significant bits) 1.203125 and 1.6015625
    x = np.array([[3, 4, 0, 0], [-3, 4, 0, 0]], np.float32)
    out, pre = orc.rmsnorm_bf16(x, np.ones(4, np.float32), 0.0)
    assert np.allclose(pre, [[1.2, 1.6, 0, 0], [-1.2, 1.6, 0, 0]], rtol=0, atol=1e-15)
    assert np.array_equal(out, np.array([[1.203125, 1.6015625, 0, 0], [-1.203125, 1.6015625, 0, 0]], np.float32))
    # a constant vector has rms |c|: the output is sign(c) * g, whatever c
    g = np.array([0.5, -2.0, 1.0, 3.0, 0.25, 1.5, -1.0, 8.0], np.float32)            # all exactly bf16
    for c in (1.0, -7.0, 1e-3, 4096.0):
        out, _ = orc.rmsnorm_bf16(np.full((1, 8), c, np.float32), g, 0.0)
        assert np.array_equal(out[0], np.sign(c) * g)
    # the gain multiplies element by element, after the division
    rng = np.random.default_rng(0)
    x = rng.standard_normal((3, 64)).astype(np.float32)
    _, p1 = orc.rmsnorm_bf16(x, np.ones(64, np.float32), 0.0)
    g = rng.uniform(0.5, 2.0, 64).astype(np.float32)
    _, pg = orc.rmsnorm_bf16(x, g, 0.0)
    assert np.allclose(pg, p1 * g.astype(np.float64), rtol=1e-15, atol=0)
    # unit mean square before the gain, and no mean subtraction: adding a constant changes the result
    assert np.allclose((p1 ** 2).mean(axis=1), 1.0, rtol=1e-12)
    _, ps = orc.rmsnorm_bf16(x + 1.0, np.ones(64, np.float32), 0.0)
    assert not np.allclose(ps, p1, atol=1e-3)


def test_rmsnorm_scale_behaviour_and_eps():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((4, 128)).astype(np.float32)
    g = rng.uniform(0.5, 2.0, 128).astype(np.float32)
    o1, p1 = orc.rmsnorm_bf16(x, g, 0.0)
    o2, p2 = orc.rmsnorm_bf16(8.0 * x, g, 0.0)                                     # power of two: exact in fp64
    assert np.array_equal(p1, p2) and np.array_equal(o1, o2)
    # eps sits under the square root beside the mean square: x / sqrt(ms + eps)
    ms = (x.astype(np.float64) ** 2).mean(axis=1, keepdims=True)
    _, pe = orc.rmsnorm_bf16(x, np.ones(128, np.float32), 0.25)
    assert np.allclose(pe, x / np.sqrt(ms + 0.25), rtol=1e-14, atol=0)
    # an all-zero token stays zero with eps > 0 (0 / sqrt(eps)) and with eps = 0 (defined as zero)
    z = np.zeros((1, 128), np.float32)
    assert not orc.rmsnorm_bf16(z, g, 1e-5)[0].any() and not orc.rmsnorm_bf16(z, g, 0.0)[0].any()


def test_rmsnorm_rounds_once_to_bf16():
    import torch
    rng = np.random.default_rng(2)
    x = rng.standard_normal((8, 256)).astype(np.float32)
    g = rng.uniform(0.5, 2.0, 256).astype(np.float32)
    out, pre = orc.rmsnorm_bf16(x, g, 1e-5)
    # every output is a bf16 value ...
    assert np.array_equal(out, torch.from_numpy(out).bfloat16().float().numpy())
    # ... the nearest one to the fp64 value (ties aside, which a random draw does not hit): the two bf16
    # neighbours of `pre` found with the library's own float -> bf16 conversion lie no closer
    lo = torch.from_numpy(pre.astype(np.float32)).bfloat16().float().numpy().astype(np.float64)
    ulp = 2.0 ** (np.floor(np.log2(np.abs(pre))) - 7)
    err = np.abs(out.astype(np.float64) - pre)
    assert np.all(err <= ulp / 2 * (1 + 1e-12))
    assert np.all(err <= np.abs(lo - pre) + 1e-300)


# ------------------------------------------------------------------ SwishGLU in front of W_down
def test_swiglu_closed_forms():
    ln3 = math.log(3.0)
    g = np.array([[0.0, ln3, -ln3, 1.0, -1.0, 40.0, -40.0, 2.5]], np.float32)
    one = np.ones_like(g)
    _, pre = orc.swiglu_bf16(g, one)
    gd = g.astype(np.float64)                                   # the oracle sees the fp32 inputs
    # sigmoid(ln 3) = 3/4 and sigmoid(-ln 3) = 1/4 (up to ln 3 having been rounded to fp32)
    assert pre[0, 0] == 0.0
    assert abs(pre[0, 1] - 0.75 * gd[0, 1]) < 1e-7 and abs(pre[0, 2] - 0.25 * gd[0, 2]) < 1e-7
    assert abs(pre[0, 3] - 0.7310585786300049) < 1e-15          # 1 / (1 + 1/e)
    # SiLU(z) - SiLU(-z) = z for every z
    assert abs((pre[0, 3] - pre[0, 4]) - 1.0) < 1e-15 and abs((pre[0, 1] - pre[0, 2]) - gd[0, 1]) < 1e-15
    # far out: the identity on the right, zero on the left
    assert abs(pre[0, 5] - 40.0) < 1e-12 and abs(pre[0, 6]) < 1e-12
    # the other operand multiplies element by element and is not passed through SiLU
    u = np.array([[2.0, -1.0, 0.5, 3.0, 0.0, 1.0, 1.0, -4.0]], np.float32)
    _, pu = orc.swiglu_bf16(g, u)
    assert np.array_equal(pu, pre * u.astype(np.float64))
    _, swapped = orc.swiglu_bf16(u, g)
    assert not np.allclose(swapped, pu)


def test_swiglu_derivative_and_single_rounding():
    import torch
    # d/dz SiLU(z) = s (1 + z (1 - s)), s = sigmoid(z): check by central differences on exactly representable points
    z = np.array([[-2.0, -0.5, 0.25, 1.5, 3.0]], np.float32)
    h = np.float32(2.0 ** -10)
    _, a = orc.swiglu_bf16(z + h, np.ones_like(z))
    _, b = orc.swiglu_bf16(z - h, np.ones_like(z))
    sgm = 1.0 / (1.0 + np.exp(-z.astype(np.float64)))
    assert np.allclose((a - b) / (2.0 * float(h)), sgm * (1.0 + z * (1.0 - sgm)), rtol=0, atol=1e-6)
    rng = np.random.default_rng(5)
    g = rng.standard_normal((4, 256)).astype(np.float32) * 2
    u = rng.standard_normal((4, 256)).astype(np.float32)
    out, pre = orc.swiglu_bf16(g, u)
    assert np.array_equal(out, torch.from_numpy(out).bfloat16().float().numpy())
    ulp = 2.0 ** (np.floor(np.log2(np.abs(pre))) - 7)
    assert np.all(np.abs(out.astype(np.float64) - pre) <= ulp / 2 * (1 + 1e-12))


# ------------------------------------------------------------------ low-bit attention states (section 3.1)
@pytest.mark.parametrize("prec", PRECS)
@pytest.mark.parametrize("case", GOLD["kv"], ids=lambda c: c["cite"][:40])
def test_kv_hand_values(case, prec):
    x = np.array([case["x"]], np.float32)
    u, v, s = orc.kv_quant(x, case["bits"], case.get("eps", EPS), prec)
    assert u[0].tolist() == case["u"]
    assert abs(s[0] - case["s"]) <= 1e-6 * max(1.0, case["s"])


@pytest.mark.parametrize("prec", PRECS)
def test_kv_at_8_bits_is_eq5_plus_the_offset(prec):
    """b = 8 must reduce to the (separately pinned) absmax INT8 quantizer of Eq. 5, head by head."""
    x = wl.rows("gauss", 91, 1, 128, 0, 96, "bf16")
    u, v, s = orc.kv_quant(x, 8, EPS, prec)
    q, v8, s8, st = orc.act_quant(x.astype(np.float64), 8, EPS, prec)
    assert np.array_equal(u.astype(np.int32) - 128, q.astype(np.int32))
    assert np.array_equal(s, s8) and np.array_equal(v, v8)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_kv_invariants(bits):
    """What the grid fixes whatever the data: the code range, the unreachable lowest code, the extreme element
    landing on the outermost level, the dequantization error bound of a symmetric grid, sign symmetry, scale
    equivariance and row independence (one statistic per head, not per token)."""
    half = 1 << (bits - 1)
    x = wl.rows("attn_out", 92, 1, 128, 0, 64, "bf16")
    u, v, s = orc.kv_quant(x, bits, EPS, 64)
    assert u.min() >= 1 and u.max() <= 2 * half - 1               # q = -2^(b-1) is never reached: |v| < 2^(b-1) - 1
    amax = np.abs(x).argmax(axis=1)
    rows = np.arange(x.shape[0])
    want_top = np.where(x[rows, amax] > 0, 2 * half - 1, 1)
    assert np.array_equal(u[rows, amax], want_top)
    deq = (u.astype(np.float64) - half) * s[:, None]
    gamma = np.abs(x).max(axis=1)
    assert np.all(np.abs(deq - x) <= 0.5 * s[:, None] + gamma[:, None] * 2e-5)   # half a step (+ the eps shrink)
    um, _, sm = orc.kv_quant(-x, bits, EPS, 64)
    assert np.array_equal(um.astype(np.int32) - half, -(u.astype(np.int32) - half)) and np.array_equal(sm, s)
    # a power-of-two rescale of one head changes that head's scale only (eps is negligible at this magnitude)
    y = x.copy(); y[3] *= 4.0
    u4, _, s4 = orc.kv_quant(y, bits, 1e-12, 64)
    u1, _, s1 = orc.kv_quant(x, bits, 1e-12, 64)
    assert np.array_equal(u4, u1) and s4[3] == 4.0 * s1[3] and np.array_equal(np.delete(s4, 3), np.delete(s1, 3))


def test_kv_mixed_widths_and_bad_arguments():
    """The [BOS] rows keep 8 bits: a per-row width must give each row exactly what a uniform call gives it."""
    x = wl.rows("gauss", 93, 1, 64, 0, 12, "bf16")
    br = np.array([8, 8, 3, 3, 3, 3, 8, 8, 3, 3, 3, 3], np.int32)
    u, v, s = orc.kv_quant(x, 3, EPS, 32, bits_row=br)
    u3, _, s3 = orc.kv_quant(x, 3, EPS, 32)
    u8, _, s8 = orc.kv_quant(x, 8, EPS, 32)
    assert np.array_equal(u[br == 3], u3[br == 3]) and np.array_equal(u[br == 8], u8[br == 8])
    assert np.array_equal(s[br == 3], s3[br == 3]) and np.array_equal(s[br == 8], s8[br == 8])
    with pytest.raises(RuntimeError):
        orc.kv_quant(x, 9, EPS, 32)
    with pytest.raises(RuntimeError):
        orc.kv_quant(x, 1, EPS, 32)
