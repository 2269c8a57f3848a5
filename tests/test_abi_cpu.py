"""CPU-only checks of the C ABI: the library builds, loads and exports what the
header declares, and argument errors are reported on the host before any launch."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2504_18415_b200 import build, hbl
    build.build()
    return hbl.lib()


def test_every_declared_symbol_is_exported(L):
    from paper_2504_18415_b200 import hbl
    header = open(os.path.join(ROOT, "include", "hbl.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(hbl_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    assert declared == set(hbl.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_size_queries(L):
    assert L.hbl_packed_weight_bytes(2048, 8192) == 2048 * 8192 // 4
    assert L.hbl_packed_weight_bytes(2040, 8192) == 0          # out_dim % 16
    assert L.hbl_packed_weight_bytes(2048, 8200) == 0          # in_dim % 128
    assert L.hbl_workspace_bytes(16, 4096, 4096) >= 16 * 4096 + 4096 * 4096
    assert L.hbl_workspace_bytes(-1, 4096, 4096) == 0
    assert L.hbl_block_workspace_bytes(16, 4096, 16384) > 0
    assert b"power of two" in L.hbl_status_string(3)


def test_argument_errors_come_before_any_launch(L):
    from paper_2504_18415_b200 import hbl
    p = C.c_void_p(1024)        # never dereferenced on the host; validation must stop first
    n = C.c_void_p(0)
    f = lambda **kw: L.hbl_forward(kw.get("x", p), kw.get("dt", 1), kw.get("T", 4), kw.get("K", 512),
                                   kw.get("W", p), kw.get("a", p), kw.get("N", 512), kw.get("bits", 4),
                                   kw.get("had", 1), kw.get("eps", 1e-5), kw.get("y", p), kw.get("ws", p),
                                   kw.get("wsb", 1 << 30), kw.get("path", 0), n)
    assert f(bits=5) == 4                      # HBL_ERR_BITS
    assert f(K=384, had=1) == 3                # HBL_ERR_NOT_POW2
    assert f(K=100) == 2                       # HBL_ERR_SHAPE
    assert f(N=100) == 2
    assert f(T=-1) == 2
    assert f(eps=0.0) == 7                     # HBL_ERR_EPS
    assert f(eps=float("nan")) == 7
    assert f(dt=7) == 10                       # HBL_ERR_FORMAT
    assert f(path=9) == 10
    assert f(T=600, path=hbl.PATH_STREAM) == 11   # HBL_ERR_TOO_LARGE
    assert f(T=600, path=hbl.PATH_STREAM_OVERLAP) == 11
    assert f(K=65536) == 11
    assert f(T=0) == 0                         # no-op
    assert f(x=n) == 1                         # HBL_ERR_NULL
    assert f(x=C.c_void_p(1028)) == 5          # HBL_ERR_ALIGN
    assert f(ws=C.c_void_p(1024 + 16)) == 5
    assert f(wsb=16) == 6                      # HBL_ERR_WORKSPACE
    q = L.hbl_quantize_weights
    assert q(n, 0, 512, 512, 1e-5, p, p, p, 1 << 20, n) == 1
    assert q(p, 0, 500, 512, 1e-5, p, p, p, 1 << 20, n) == 2
    assert q(p, 0, 512, 512, -1.0, p, p, p, 1 << 20, n) == 7
    assert q(p, 0, 512, 512, 1e-5, p, p, p, 8, n) == 6
    assert L.hbl_hadamard_f32(p, 0, 4, 384, p, n) == 3
    assert L.hbl_norm_quantize_act(p, p, 0, -1.0, 4, 4096, 4, 1e-5, p, p, p, n, n) == 7   # norm_eps < 0
    assert L.hbl_norm_quantize_act(p, n, 0, 1e-5, 4, 4096, 4, 1e-5, p, p, p, n, n) == 1   # no gain
    assert L.hbl_norm_quantize_act(p, p, 5, 1e-5, 4, 4096, 4, 1e-5, p, p, p, n, n) == 10  # gain dtype
    assert L.hbl_norm_quantize_act(p, p, 1, 1e-5, 4, 1024, 4, 1e-5, p, p, p, n, n) == 2   # width without a fused kernel
    assert L.hbl_forward_norm(p, p, 0, 1e-5, 4, 384, p, p, 512, 4, 1e-5, p, p, 1 << 30, 0, n) == 3
    assert L.hbl_glu_quantize_act(p, n, 4, 4096, 4, 1e-5, p, p, p, n, n) == 1             # no `up`
    assert L.hbl_glu_quantize_act(p, p, 4, 1024, 4, 1e-5, p, p, p, n, n) == 2
    assert L.hbl_forward_glu(p, p, 4, 384, p, p, 512, 4, 1e-5, p, p, 1 << 30, 0, n) == 3
    qr = L.hbl_quantize_weights_rotated
    assert qr(p, 0, 512, 384, 1e-5, p, p, p, 1 << 30, n) == 3                                # W H needs in_dim = 2^m
    assert qr(p, 0, 512, 512, 1e-5, p, p, p, 1 << 16, n) == 6                                # no room for the fp32 copy of W H
    assert L.hbl_quantize_weights_rotated_workspace_bytes(512, 512) >= 4 * 512 * 512
    assert L.hbl_hadamard_bf16(p, 4, 384, p, n) == 3             # not a power of two
    assert L.hbl_hadamard_bf16(p, 4, 1024, p, n) == 2            # outside 2048..16384
    assert L.hbl_hadamard_bf16(n, 4, 4096, p, n) == 1
    assert L.hbl_hadamard_bf16(p, 0, 4096, p, n) == 0            # no tokens: no-op
    assert L.hbl_quantize_act(p, 0, 4, 512, 3, 1, 1e-5, p, p, p, n) == 4
    assert L.hbl_gemm_i32(p, n, 4, 512, p, 512, p, p, 1 << 30, hbl.PATH_STREAM, n) == 1   # codesum required
    assert L.hbl_gemm_i32(p, p, 4, 512, p, 512, p, p, 1 << 30, hbl.PATH_STREAM_OVERLAP, n) == 10   # quantizing calls only
    kv = lambda **kw: L.hbl_quantize_kv(kw.get("x", p), kw.get("T", 4), kw.get("H", 8), kw.get("D", 128), kw.get("bits", 4),
                                        kw.get("S", 0), kw.get("eps", 1e-5), kw.get("codes", p), kw.get("scale", p),
                                        kw.get("bos", n), kw.get("bos_scale", n), n)
    assert kv(bits=5) == 4 and kv(bits=2) == 4
    assert kv(D=96) == 2 and kv(H=0) == 2 and kv(T=-1) == 2
    assert kv(eps=0.0) == 7
    assert kv(bos=p, bos_scale=p, S=0) == 2                     # [BOS] rows asked for without a sequence length
    assert kv(bos=p, S=16) == 1                                 # ... without their scales
    assert kv(x=n) == 1 and kv(x=C.c_void_p(1032)) == 5
    assert kv(T=0) == 0
    L.hbl_kv_codes_bytes.restype = C.c_size_t
    assert L.hbl_kv_codes_bytes(10, 8, 128, 3) == 10 * 8 * 48 and L.hbl_kv_codes_bytes(10, 8, 100, 4) == 0
    b = hbl.hbl_block_t()
    b.tokens, b.hidden, b.ffn, b.bits, b.x_dtype, b.eps = 4, 4096, 12288, 4, 1, 1e-5
    assert L.hbl_block_forward(C.byref(b), p, 1 << 40, 0, n) == 3                         # ffn not 2^m
    b.ffn = 16384
    assert L.hbl_block_forward(C.byref(b), p, 1 << 40, 0, n) == 1                         # null inputs
    assert L.hbl_block_forward(None, p, 1 << 40, 0, n) == 1


def test_product_path_has_no_cpu_fallback():
    """The binding must not import the oracle, and must fail loudly without the library."""
    src = open(os.path.join(ROOT, "paper_2504_18415_b200", "hbl.py")).read()
    assert "oracle" not in src.replace("no CPU\nfallback", "")
    for f in os.listdir(os.path.join(ROOT, "paper_2504_18415_b200", "csrc")):
        assert "oracle" not in open(os.path.join(ROOT, "paper_2504_18415_b200", "csrc", f)).read()
