"""GPU parity of the quantize-and-pack step (Eq. 6, two INT4 codes per byte) and of the contraction that widens them.

The packed bytes are decoded here, on the host, from the layout the header documents; the decoded codes must be
the ones hbl_quantize_act gives (bit for bit) and obey the usual rule against the oracle; the contraction on packed
codes must give the oracle's exact integers."""
import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS, check_codes, check_y, oracle_layer, to_dev

pytestmark = pytest.mark.gpu


def decode(packed: np.ndarray) -> np.ndarray:
    """[T, K/2] bytes -> [T, K] codes: word g covers elements 8g..8g+7, byte b = (q[8g+b]+8) | (q[8g+b+4]+8) << 4."""
    T, half = packed.shape
    w = packed.reshape(T, half // 4, 4)
    out = np.empty((T, half // 4, 8), dtype=np.int8)
    out[:, :, 0:4] = (w & 15).astype(np.int8) - 8
    out[:, :, 4:8] = (w >> 4).astype(np.int8) - 8
    return out.reshape(T, 2 * half)


def encode(q: np.ndarray) -> np.ndarray:
    T, K = q.shape
    u = (q.astype(np.int16) + 8).astype(np.uint8).reshape(T, K // 8, 8)
    return (u[:, :, 0:4] | (u[:, :, 4:8] << 4)).reshape(T, K // 2)


@pytest.mark.parametrize("K,had", [(2048, True), (4096, True), (8192, True), (16384, True), (4096, False), (1152, False),
                                   (11008, False)])
def test_packed_codes_match_unpacked_and_oracle(K, had):
    T = 131 if K <= 8192 else 67
    kind = "ffn_mid" if K >= 8192 else "attn_out"
    x = wl.rows(kind, 40 + K, 1, K, 0, T, "bf16")
    xd = to_dev(x, "bf16")
    pk, scale = hbl.hbl_quantize_act_int4_packed(xd, had, EPS)
    codes, scale1, _ = hbl.hbl_quantize_act(xd, 4, had, EPS)
    assert hbl.hbl_check_status() == 0
    got = decode(pk.cpu().numpy())
    assert np.array_equal(got, codes.cpu().numpy())
    assert torch.equal(scale, scale1)
    xr = orc.hadamard(x) if had else x.astype(np.float64)
    q, v, s, st = orc.act_quant(xr, 4, EPS, 32)
    check_codes(got, q, v)
    assert got.min() >= -8 and got.max() <= 7


@pytest.mark.parametrize("T,K,N", [(1, 128, 16), (130, 1024, 784), (257, 2048, 2048), (1000, 8192, 528), (4096, 4096, 4096)])
def test_contraction_on_packed_codes_is_exact(T, K, N):
    rng = np.random.default_rng(T + K + N)
    q = rng.integers(-8, 8, size=(T, K), dtype=np.int8)
    q[0, :] = -8; q[-1, :] = 7                                  # the extreme codes in whole rows
    W = wl.rows("latent", 77, 61, K, 0, N, "f32")
    packed, _ = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    pk = torch.from_numpy(encode(q)).cuda()
    acc = hbl.hbl_gemm_i32_int4_packed(pk, packed, N)
    assert hbl.hbl_check_status() == 0
    ref = hbl.hbl_gemm_i32(torch.from_numpy(q).cuda(), None, packed, N, hbl.PATH_TENSOR)
    assert torch.equal(acc, ref)
    if T * K * N <= 3e9:
        wt = hbl.hbl_unpack_weights(packed, N, K).cpu().numpy()
        assert np.array_equal(acc.cpu().numpy(), orc.gemm(q, wt))


def test_packed_entry_points_refuse_what_they_cannot_do():
    L = hbl.lib()
    x = torch.zeros((8, 1024), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((8, 512), dtype=torch.uint8, device="cuda")
    sc = torch.zeros((8,), dtype=torch.float32, device="cuda")
    call = lambda dt, T, K, had: L.hbl_quantize_act_int4_packed(x.data_ptr(), dt, T, K, had, EPS, out.data_ptr(), sc.data_ptr(), None)
    assert call(1, 8, 1024, 1) == 2          # no packing kernel for this width with the transform
    assert call(0, 100, 4096, 1) == 2        # fp32 input
    assert call(1, 8, 1024, 0) == 2          # 64 tokens or fewer without the transform
    assert call(1, 0, 4096, 1) == 0


@pytest.mark.parametrize("cfg,T", [(wl.CONFIG2, 300), (wl.CONFIG3, 1024), (wl.CONFIG3, 4224)],
                         ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_layer_with_packed_codes_equals_the_plain_path_and_the_oracle(cfg, T):
    """The whole layer with the codes packed between its two kernels: the same integers are contracted, so the
    result must equal the one-code-per-byte path bit for bit, and the oracle within the usual bar."""
    rows = min(T, 1024)
    x_rows = cfg.x(0, rows)
    W = cfg.w_latent()
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    x = to_dev(x_rows, "bf16")
    if rows < T:
        x = x.repeat((T + rows - 1) // rows, 1)[:T].contiguous()
    y = hbl.hbl_forward(x, packed, alpha, cfg.N, 4, True, EPS, path=hbl.PATH_TENSOR_PACKED)
    ref = hbl.hbl_forward(x, packed, alpha, cfg.N, 4, True, EPS, path=hbl.PATH_TENSOR)
    assert hbl.hbl_check_status() == 0
    assert torch.equal(y, ref)
    toks = [0, 127, 128, rows - 1]
    o = oracle_layer(x_rows[toks], W, 4, True)
    check_y(y[toks], o["y64"])


def test_block_with_packed_codes_equals_the_plain_path():
    H, F, T = 2048, 8192, 700
    seed = 33
    g = torch.Generator(device="cuda").manual_seed(seed)
    ins = {"attn_in": to_dev(wl.rows("gauss", seed, 10, H, 0, T, "bf16"), "bf16"), "o_in": to_dev(wl.rows("attn_out", seed, 11, H, 0, T, "bf16"), "bf16"),
           "ffn_in": to_dev(wl.rows("gauss", seed, 12, H, 0, T, "bf16"), "bf16")}      # no down_in: the call chains the gating product
    shapes = {"q": (H, H), "k": (H, H), "v": (H, H), "o": (H, H), "up": (F, H), "gate": (F, H), "down": (H, F)}
    packed, alphas = {}, []
    for n, (N, K) in shapes.items():
        p, a = hbl.hbl_quantize_weights(torch.randn((N, K), device="cuda", generator=g) * 0.02, EPS)
        packed[n] = p; alphas.append(a)
    alpha7 = torch.cat(alphas)
    a = hbl.hbl_block_forward(ins, packed, alpha7, H, F, 4, EPS, path=hbl.PATH_TENSOR_PACKED)
    a = {n: v.clone() for n, v in a.items()}
    b = hbl.hbl_block_forward(ins, packed, alpha7, H, F, 4, EPS, path=hbl.PATH_TENSOR)
    assert hbl.hbl_check_status() == 0
    for n in shapes:
        assert torch.equal(a[n], b[n]), n


def test_packed_path_argument_errors():
    L = hbl.lib()
    p = 1024
    f = lambda bits, dt, K, had: L.hbl_forward(p, dt, 300, K, p, p, 512, bits, had, EPS, p, p, 1 << 40, hbl.PATH_TENSOR_PACKED, None)
    assert f(8, 1, 4096, 1) == 2           # INT8 codes are not packed
    assert f(4, 0, 4096, 1) == 2           # fp32 input: no packing kernel
    assert f(4, 1, 1024, 1) == 2           # width without one
    assert L.hbl_gemm_i32(p, None, 300, 1024, p, 512, p, p, 1 << 40, hbl.PATH_TENSOR_PACKED, None) == 10
