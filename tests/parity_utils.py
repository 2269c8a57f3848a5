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


def check_codes(q_gpu: np.ndarray, q_orc: np.ndarray, v_orc: np.ndarray, max_frac=1e-4, near=1e-5):
    diff = q_gpu.astype(np.int32) - q_orc.astype(np.int32)
    bad = np.nonzero(diff)
    n_bad = len(bad[0])
    assert n_bad <= max(1, int(max_frac * q_orc.size)), f"{n_bad} of {q_orc.size} codes differ"
    if n_bad:
        d = diff[bad]
        assert np.all(np.abs(d) == 1), "a code differs by more than 1"
        b = q_orc[bad].astype(np.float64) + 0.5 * d          # boundary between the two codes
        dist = np.abs(v_orc[bad] - b)
        assert np.all(dist <= near * np.maximum(1.0, np.abs(b))), f"flip away from a boundary: {dist.max()}"
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


def reconcile_bf16_inputs(xr_gpu: torch.Tensor, x_orc: np.ndarray, pre: np.ndarray, rel=4e-6):
    """For the entry points that form the transform's bf16 input on the fly (normalisation, gating product).

    The oracle forms that input in fp64 and rounds it once to bf16; the kernel forms it in fp32.  The rounding
    is a decision, and where the exact value lies within the kernel's evaluation error of the midpoint between
    two bf16 values the kernel may take it the other way; when that element is large, a visible share of the
    token's codes follows it.  So the decision is checked on its own and everything after it is compared given
    the kernel's decisions:
      * the kernel's input is recovered from its exported transform (the transform is its own inverse);
      * every element must be the oracle's bf16 value, or the neighbouring one with the exact value `pre`
        within `rel` (relative) of the midpoint between the two;
      * returned: the kernel's input as bf16-valued fp32, for the oracle's later stages, and how many
        elements were rounded the other way."""
    rec = orc.hadamard(xr_gpu.float().cpu().numpy())
    noise = 2e-5 * np.abs(rec).max(axis=1, keepdims=True)            # accuracy of the recovery (fp32 export)
    a = np.abs(x_orc).astype(np.float64)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(a, 2.0 ** -100))) - 7)
    diff = rec - x_orc
    moved = np.abs(diff) > np.maximum(0.5 * ulp, 4 * noise)
    x_gpu = x_orc.copy()
    if moved.any():
        ratio = np.abs(diff[moved]) / ulp[moved]
        # one bf16 step away (half a step when the value sits on a power of two and the step goes down)
        assert np.all((np.abs(ratio - 1.0) <= 0.3) | (np.abs(ratio - 0.5) <= 0.15)), "an input is off by more than one bf16 step"
        target = x_orc[moved].astype(np.float64) + np.sign(diff[moved]) * np.where(ratio > 0.75, 1.0, 0.5) * ulp[moved]
        nb = torch.from_numpy(target.astype(np.float32)).bfloat16().float().numpy()
        mid = 0.5 * (x_orc[moved].astype(np.float64) + nb)
        assert np.all(np.abs(pre[moved] - mid) <= rel * np.abs(pre[moved])), "an input was rounded the other way, away from a midpoint"
        x_gpu[moved] = nb
    return x_gpu, int(moved.sum())
