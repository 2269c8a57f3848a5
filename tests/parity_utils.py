"""Shared helpers of the GPU parity tests: tolerance rules and the oracle calls.

Tolerances (the layer's stated bars):
  * integer work (ternary weights given alpha, int32 accumulators given codes): bit-exact;
  * Hadamard outputs: |dx_r| <= 1e-5 * max_k |x_r[t,:]| (fp32 butterflies vs the fp64 oracle);
  * codes: at most 1e-4 of them may differ from the oracle's, each by +-1 and only where the
    oracle's pre-rounding value v lies within 1e-5 * max(1, |b|) of the rounding boundary b
    between the two codes (both sides take the decision in fp32; the only difference left is
    the rounding order of the fp32 butterflies and of the per-token sum);
  * bf16 outputs: |dy| <= 1e-2 * max(|y|, rms of the token's row).
"""
import numpy as np
import torch

from oracle import hbl_oracle as orc

EPS = 1e-5


def to_dev(x_f32: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x_f32)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t      # values are bf16-exact: lossless


def check_codes(q_gpu: np.ndarray, q_orc: np.ndarray, v_orc: np.ndarray, max_frac=1e-4):
    diff = q_gpu.astype(np.int32) - q_orc.astype(np.int32)
    bad = np.nonzero(diff)
    n_bad = len(bad[0])
    assert n_bad <= max(1, int(max_frac * q_orc.size)), f"{n_bad} of {q_orc.size} codes differ"
    if n_bad:
        d = diff[bad]
        assert np.all(np.abs(d) == 1), "a code differs by more than 1"
        b = q_orc[bad].astype(np.float64) + 0.5 * d          # boundary between the two codes
        dist = np.abs(v_orc[bad] - b)
        assert np.all(dist <= 1e-5 * np.maximum(1.0, np.abs(b))), f"flip away from a boundary: {dist.max()}"
    return n_bad


def check_y(y_gpu_bf16: torch.Tensor, y64: np.ndarray, rel=1e-2):
    y = y_gpu_bf16.float().cpu().numpy().astype(np.float64)
    rms = np.sqrt((y64 ** 2).mean(axis=1, keepdims=True))
    tol = rel * np.maximum(np.abs(y64), rms)
    err = np.abs(y - y64)
    assert np.all(err <= tol + 1e-30), f"max err/tol = {(err / (tol + 1e-30)).max()}"


def oracle_layer(x_f32, W_f32, bits, had, eps=EPS):
    """Everything the oracle can say about one layer call."""
    wt, alpha = orc.weight_quant(W_f32, eps, 32)
    xr = orc.hadamard(x_f32) if had else x_f32.astype(np.float64)
    q, v, s, st = orc.act_quant(xr, bits, eps, 32)
    acc = orc.gemm(q, wt)
    yb, y64 = orc.rescale(acc, s, alpha)
    return dict(wt=wt, alpha=alpha, xr=xr, q=q, v=v, s=s, acc=acc, y_bits=yb, y64=y64)
