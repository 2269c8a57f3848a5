"""Seeded synthetic inputs for the H-BitLinear forward path.

This module only *draws inputs*: it holds none of the layer's arithmetic (no
transform, no quantizer, no contraction).  Both the CUDA path's callers and the
CPU oracle's callers take their tensors from here, so the two sides see the
same bits.

Every tensor is generated in independent blocks of ``ROWS_PER_BLOCK`` rows from
a counter-based generator (numpy Philox) keyed by ``(seed, tensor_id, block)``,
so any row range can be produced without generating what comes before it and
large tensors can be drawn by several threads.

Activations are returned in their storage dtype's exact values, as fp32 arrays
(bf16 activations are fp32 values whose low 16 bits are zero) together with the
raw bf16 bit pattern when asked for.

Workload recipes (the paper gives only model shapes, Table 8, and a qualitative
picture of the activations in section 2.1: Gaussian-like inputs to W_qkv and
W_up,gate; outlier channels plus a mass of entries near zero in the inputs of
W_o and W_down):

  gauss        N(0,1)
  outlier50    N(0,1), a seeded 1 % of channels multiplied by 50
  attn_out     N(0,1) + Student-t(3) added on a seeded 5 % of entries, then a
               seeded 0.5 % of channels multiplied by 30        (W_o input)
  ffn_mid      SiLU(a)*b with a,b iid N(0,1), then a seeded 0.2 % of channels
               multiplied by 40                                 (W_down input)
  latent weights  N(0, 0.02^2) in fp32
"""
from __future__ import annotations

import concurrent.futures as _cf
import os
from dataclasses import dataclass

import numpy as np

ROWS_PER_BLOCK = 64
_CHANNEL_BLOCK = (1 << 62)          # block id reserved for per-tensor channel draws


def _rng(seed: int, tensor_id: int, block: int) -> np.random.Generator:
    key = [((int(seed) & 0xFFFFFFFF) << 32) | (int(tensor_id) & 0xFFFFFFFF), int(block)]
    return np.random.Generator(np.random.Philox(key=key))


def round_to_bf16(x: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Round fp32 -> bf16 (nearest even).  Returns (fp32 values, uint16 bits)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
    back = (r.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return back.reshape(x.shape), r.reshape(x.shape)


def outlier_channels(seed: int, tensor_id: int, K: int, fraction: float) -> np.ndarray:
    """The seeded set of outlier channels of one tensor (sorted indices)."""
    n = max(1, int(round(K * fraction)))
    g = _rng(seed, tensor_id, _CHANNEL_BLOCK)
    return np.sort(g.choice(K, size=n, replace=False))


def _block_rows(kind: str, seed: int, tensor_id: int, K: int, block: int) -> np.ndarray:
    g = _rng(seed, tensor_id, block)
    R = ROWS_PER_BLOCK
    if kind == "gauss":
        x = g.standard_normal((R, K), dtype=np.float32)
    elif kind == "outlier50":
        x = g.standard_normal((R, K), dtype=np.float32)
        x[:, outlier_channels(seed, tensor_id, K, 0.01)] *= np.float32(50.0)
    elif kind == "attn_out":
        x = g.standard_normal((R, K), dtype=np.float32)
        mask = g.random((R, K), dtype=np.float32) < np.float32(0.05)
        t3 = g.standard_t(3.0, size=(R, K)).astype(np.float32)
        x = x + np.where(mask, t3, np.float32(0.0))
        x[:, outlier_channels(seed, tensor_id, K, 0.005)] *= np.float32(30.0)
    elif kind == "ffn_mid":
        a = g.standard_normal((R, K), dtype=np.float32)
        b = g.standard_normal((R, K), dtype=np.float32)
        x = (a / (np.float32(1.0) + np.exp(-a))) * b
        x[:, outlier_channels(seed, tensor_id, K, 0.002)] *= np.float32(40.0)
    elif kind == "latent":
        x = g.standard_normal((R, K), dtype=np.float32) * np.float32(0.02)
    else:
        raise ValueError(f"unknown workload kind {kind!r}")
    return np.ascontiguousarray(x, dtype=np.float32)


def rows(kind: str, seed: int, tensor_id: int, K: int, row0: int, nrows: int,
         dtype: str = "f32", threads: int | None = None) -> np.ndarray:
    """Rows [row0, row0+nrows) of the tensor, as fp32 values exact in `dtype`."""
    if nrows == 0:
        return np.zeros((0, K), dtype=np.float32)
    b0 = row0 // ROWS_PER_BLOCK
    b1 = (row0 + nrows - 1) // ROWS_PER_BLOCK
    out = np.empty(((b1 - b0 + 1) * ROWS_PER_BLOCK, K), dtype=np.float32)

    def work(b):
        blk = _block_rows(kind, seed, tensor_id, K, b)
        if dtype == "bf16":
            blk, _ = round_to_bf16(blk)
        out[(b - b0) * ROWS_PER_BLOCK:(b - b0 + 1) * ROWS_PER_BLOCK] = blk

    nthr = threads or min(32, os.cpu_count() or 1)
    blocks = range(b0, b1 + 1)
    if nthr > 1 and len(blocks) > 1:
        with _cf.ThreadPoolExecutor(nthr) as ex:
            list(ex.map(work, blocks))
    else:
        for b in blocks:
            work(b)
    lo = row0 - b0 * ROWS_PER_BLOCK
    return out[lo:lo + nrows]


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of fp32 values that are already exact in bf16."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    assert not np.any(u & np.uint32(0xFFFF)), "values are not exact in bf16"
    return (u >> np.uint32(16)).astype(np.uint16)


# ----------------------------------------------------------------------------
# The five workload configurations.
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class LayerWorkload:
    name: str
    seed: int
    K: int                 # in_dim
    N: int                 # out_dim
    bits: int              # 4 | 8
    use_hadamard: bool
    x_kind: str
    x_dtype: str           # "f32" | "bf16"
    tokens: tuple          # the token counts of the sweep
    x_id: int = 1
    w_id: int = 2

    def x(self, row0: int, nrows: int) -> np.ndarray:
        return rows(self.x_kind, self.seed, self.x_id, self.K, row0, nrows, self.x_dtype)

    def w_latent(self, row0: int = 0, nrows: int | None = None) -> np.ndarray:
        n = self.N if nrows is None else nrows
        return rows("latent", self.seed, self.w_id, self.K, row0, n, "f32")


CONFIG1 = LayerWorkload("config1", 0, 512, 512, 4, True, "outlier50", "f32", (64,))
CONFIG2 = LayerWorkload("config2_Wo_1p3B", 2, 2048, 2048, 4, True, "attn_out", "bf16", (1, 16, 256, 4096))
CONFIG3 = LayerWorkload("config3_Wdown_1p3B", 3, 8192, 2048, 4, True, "ffn_mid", "bf16", (1, 16, 1024, 16384))
CONFIG4A = LayerWorkload("config4_a8_N12288", 4, 4096, 12288, 8, False, "gauss", "bf16", (16, 4096, 32768))
CONFIG4B = LayerWorkload("config4_a8_N32768", 4, 4096, 32768, 8, False, "gauss", "bf16", (16, 4096, 32768), w_id=3)
LAYER_CONFIGS = (CONFIG1, CONFIG2, CONFIG3, CONFIG4A, CONFIG4B)


@dataclass(frozen=True)
class BlockWorkload:
    """7B-shaped decoder block: the seven projections on caller-supplied inputs."""
    name: str = "config5_block_7B"
    seed: int = 5
    hidden: int = 4096
    ffn: int = 16384
    bits: int = 4
    x_dtype: str = "bf16"
    tokens: tuple = (1, 4, 16, 64, 256, 1024, 4096, 16384, 65536)

    # tensor ids: inputs 10..13, weights 20..26 (q,k,v,o,up,gate,down)
    def x_attn_in(self, r0, n): return rows("gauss", self.seed, 10, self.hidden, r0, n, self.x_dtype)
    def x_o_in(self, r0, n): return rows("attn_out", self.seed, 11, self.hidden, r0, n, self.x_dtype)
    def x_ffn_in(self, r0, n): return rows("gauss", self.seed, 12, self.hidden, r0, n, self.x_dtype)
    def x_down_in(self, r0, n): return rows("ffn_mid", self.seed, 13, self.ffn, r0, n, self.x_dtype)

    def weight_shapes(self):
        H, F = self.hidden, self.ffn
        return {"q": (H, H), "k": (H, H), "v": (H, H), "o": (H, H),
                "up": (F, H), "gate": (F, H), "down": (H, F)}

    def w_latent(self, which: str, row0: int = 0, nrows: int | None = None) -> np.ndarray:
        names = ["q", "k", "v", "o", "up", "gate", "down"]
        N, K = self.weight_shapes()[which]
        n = N if nrows is None else nrows
        return rows("latent", self.seed, 20 + names.index(which), K, row0, n, "f32")


CONFIG5 = BlockWorkload()
