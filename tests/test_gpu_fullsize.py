"""GPU parity at the benchmark's full sizes, in the launch configuration the benchmark times.

The oracle cannot redo 16384 x 8192 x 2048 in seconds, but every token is independent (Eq. 3-7 work row
by row), so the GPU runs the whole batch and the oracle recomputes a sample of its tokens -- every output
of each sampled token -- from the same inputs.  As in the benchmark, batches beyond 4096 tokens tile a
seeded block of 4096 rows; the sample takes tokens from different tiles, from both ends of a 128-token
tile of the contraction, and the last token; every 4096-row replica must repeat the first one bit for bit,
which covers every token tile of the batch."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS, check_codes, check_y, oracle_layer, to_dev

pytestmark = pytest.mark.gpu

HOST_ROWS = 4096


def batch(x_rows: np.ndarray, T: int, dtype: str) -> torch.Tensor:
    x = to_dev(x_rows, dtype)
    if x.shape[0] < T:
        x = x.repeat((T + x.shape[0] - 1) // x.shape[0], 1)[:T].contiguous()
    return x


def sample_tokens(T: int):
    cand = [0, 1, 127, 128, 129, T // 3, HOST_ROWS - 1, HOST_ROWS, 2 * HOST_ROWS + 77, T - 130, T - 2, T - 1]
    return sorted({t for t in cand if 0 <= t < T})


def check_replicas(y: torch.Tensor, rows: int):
    """Tokens that repeat a seeded row must repeat its output exactly, wherever they sit in the batch."""
    T = y.shape[0]
    for r0 in range(rows, T, rows):
        n = min(rows, T - r0)
        assert torch.equal(y[r0:r0 + n], y[:n]), f"replica at row {r0} differs from the first {n} rows"


# config 2 and 3: every token count of their sweeps; config 4 (both widths): its sweep plus the sizes at which a
# single layer changes kernel (160 tokens: 32 MiB of packed weights still stream; 4096: the large-batch kernel)
@pytest.mark.parametrize("cfg,T", [(wl.CONFIG3, 16384), (wl.CONFIG3, 1024), (wl.CONFIG3, 16), (wl.CONFIG3, 1),
                                   (wl.CONFIG2, 4096), (wl.CONFIG2, 256), (wl.CONFIG2, 16), (wl.CONFIG2, 1),
                                   (wl.CONFIG4A, 32768), (wl.CONFIG4A, 4096), (wl.CONFIG4A, 16),
                                   (wl.CONFIG4B, 32768), (wl.CONFIG4B, 4096), (wl.CONFIG4B, 160), (wl.CONFIG4B, 16)],
                         ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_layer_full_size_sampled_tokens(cfg, T):
    rows = min(T, HOST_ROWS)
    x_rows = cfg.x(0, rows)
    W = cfg.w_latent()
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    y = hbl.hbl_forward(batch(x_rows, T, cfg.x_dtype), packed, alpha, cfg.N, cfg.bits, cfg.use_hadamard, EPS)
    assert hbl.hbl_check_status() == 0
    toks = sample_tokens(T)
    o = oracle_layer(x_rows[[t % rows for t in toks]], W, cfg.bits, cfg.use_hadamard)
    assert alpha.item() == o["alpha"]
    check_y(y[toks], o["y64"])
    check_replicas(y, rows)


# ---- the 7B-shaped decoder block (config 5) at every token count of its sweep and at the sizes where
#      hbl_block_forward changes its launch configuration ----
BLOCK_SRC = {"q": "attn_in", "k": "attn_in", "v": "attn_in", "o": "o_in", "up": "ffn_in", "gate": "ffn_in",
             "down": "down_in"}


@pytest.fixture(scope="module")
def block7b():
    """Weights of the block, ternarised once by the library and once by the oracle (compared), and the seeded
    4096-row input blocks."""
    cfg = wl.CONFIG5
    packed, alphas, wt, al = {}, [], {}, {}
    for n in cfg.weight_shapes():
        lat = cfg.w_latent(n)
        p, a = hbl.hbl_quantize_weights(torch.from_numpy(lat).cuda(), EPS)
        wt[n], al[n] = orc.weight_quant(lat, EPS, 32)
        assert a.item() == al[n]
        packed[n] = p
        alphas.append(a)
        del lat
    xin = {"attn_in": cfg.x_attn_in(0, HOST_ROWS), "o_in": cfg.x_o_in(0, HOST_ROWS),
           "ffn_in": cfg.x_ffn_in(0, HOST_ROWS), "down_in": cfg.x_down_in(0, HOST_ROWS)}
    return dict(cfg=cfg, packed=packed, alpha7=torch.cat(alphas), wt=wt, al=al, xin=xin)


def oracle_rows(b, name, rows_idx):
    """All outputs of projection `name` for the given rows of its seeded input block."""
    x = b["xin"][BLOCK_SRC[name]][rows_idx]
    xr = orc.hadamard(x) if name in ("o", "down") else x.astype(np.float64)
    q, v, s, st = orc.act_quant(xr, b["cfg"].bits, EPS, 32)
    return orc.rescale(orc.gemm(q, b["wt"][name]), s, b["al"][name])[1]


# 1 ... 65536 in powers of 4 is the sweep; 129 / 512 are the first and last multi-pass sizes of the streaming
# launch (seven weight tensors, four inputs, passes of 128 tokens), 513 the first size on the large-batch kernel
@pytest.mark.parametrize("T", [1, 4, 16, 64, 129, 256, 512, 513, 1024, 4096, 16384, 65536])
def test_block_full_size_sampled_tokens(block7b, T):
    b = block7b
    cfg = b["cfg"]
    H, F = cfg.hidden, cfg.ffn
    rows = min(T, HOST_ROWS)
    ins = {k: batch(v[:rows], T, cfg.x_dtype) for k, v in b["xin"].items()}
    outs = hbl.hbl_block_forward(ins, b["packed"], b["alpha7"], H, F, cfg.bits, EPS)
    assert hbl.hbl_check_status() == 0
    cand = [0, 5, 127, 128, 129, 255, 256, 383, 384, 511, 512, T // 2 + 3, HOST_ROWS + 130, T - 129, T - 1]
    toks = sorted({t for t in cand if 0 <= t < T})
    for n in cfg.weight_shapes():
        check_y(outs[n][toks], oracle_rows(b, n, [t % rows for t in toks]))
        check_replicas(outs[n], rows)
    if T in (256, 512):
        # the multi-pass streaming launch and the large-batch kernel contract the same integers and round once
        ref = hbl.hbl_block_forward(ins, b["packed"], b["alpha7"], H, F, cfg.bits, EPS, path=hbl.PATH_TENSOR)
        assert hbl.hbl_check_status() == 0
        for n in cfg.weight_shapes():
            assert torch.equal(outs[n], ref[n]), f"{n}: streaming and large-batch kernels differ at {T} tokens"


@pytest.mark.parametrize("T", [1024, 16384])
def test_block_full_size_sampled_output_columns(block7b, T):
    """The other cut through a full-size result: a few output columns of every projection over ALL tokens of the
    seeded block (the contraction redone by the oracle for those weight rows only).

    Over thousands of tokens a few codes do sit on a rounding boundary, and a token with two of them moves its
    small outputs by more than 1e-2 of the row's rms although every code obeys its own rule.  So the two bars are
    checked one after the other: the codes of all tokens against the oracle's (at most 1e-4 of them one step
    away, each within 1e-5 of a boundary), then the outputs against the oracle's contraction and rescale of
    the codes the GPU decided on."""
    b = block7b
    cfg = b["cfg"]
    H, F = cfg.hidden, cfg.ffn
    rows = min(T, HOST_ROWS)
    ins = {k: batch(v[:rows], T, cfg.x_dtype) for k, v in b["xin"].items()}
    outs = hbl.hbl_block_forward(ins, b["packed"], b["alpha7"], H, F, cfg.bits, EPS)
    assert hbl.hbl_check_status() == 0
    quant = {}
    for n, (N, K) in cfg.weight_shapes().items():
        src = BLOCK_SRC[n]
        had = n in ("o", "down")
        if src not in quant:
            x = b["xin"][src][:rows]
            xr = orc.hadamard(x) if had else x.astype(np.float64)
            q, v, s, st = orc.act_quant(xr, cfg.bits, EPS, 32)
            codes, scale, _ = hbl.hbl_quantize_act(ins[src][:rows].contiguous(), cfg.bits, had, EPS)
            qg = codes.cpu().numpy()
            check_codes(qg, q, v)
            assert np.allclose(scale.cpu().numpy(), s, rtol=2e-6, atol=0)
            quant[src] = (qg, s)
        qg, s = quant[src]
        cols = sorted({0, 127, 128, 255, 256, N // 2 + 1, N - 129, N - 1})
        y64 = orc.rescale(orc.gemm(qg, b["wt"][n][cols]), s, b["al"][n])[1]
        got = outs[n][:rows][:, cols].float().cpu().numpy().astype(np.float64)
        # The bar is 1e-2 of max(|y|, rms of the token's output row).  The whole row is not recomputed here, so
        # its rms is taken from the operands: over weight rows, sum_k w q has mean square mean(w^2) * sum_k q^2
        # (ternary entries, independent of the codes), times the row's alpha * s_t.
        w2 = float((b["wt"][n].astype(np.float64) ** 2).mean())
        rms = float(b["al"][n]) * s * np.sqrt(w2 * (qg.astype(np.float64) ** 2).sum(axis=1))
        tol = 1e-2 * np.maximum(np.abs(y64), rms[:, None])
        assert np.all(np.abs(got - y64) <= tol), f"{n}: max err/tol {(np.abs(got - y64) / tol).max()}"
