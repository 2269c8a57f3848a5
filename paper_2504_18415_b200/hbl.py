"""Thin Python binding of libhbl.so (the C ABI in include/hbl.h).

Argument marshalling only: every step of the layer runs in the library's CUDA
kernels.  torch is used for device memory and streams.  There is no CPU
fallback: if the library is missing or cannot be loaded, importing a function
from here raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

HBL_OK = 0
HBL_F32, HBL_BF16 = 0, 1
PATH_AUTO, PATH_STREAM, PATH_TENSOR, PATH_TENSOR_PACKED, PATH_STREAM_OVERLAP = 0, 1, 2, 3, 4

STATUS_NAMES = {
    0: "HBL_OK", 1: "HBL_ERR_NULL", 2: "HBL_ERR_SHAPE", 3: "HBL_ERR_NOT_POW2", 4: "HBL_ERR_BITS",
    5: "HBL_ERR_ALIGN", 6: "HBL_ERR_WORKSPACE", 7: "HBL_ERR_EPS", 8: "HBL_ERR_CUDA", 9: "HBL_ERR_TIMEOUT",
    10: "HBL_ERR_FORMAT", 11: "HBL_ERR_TOO_LARGE",
}

EXPORTS = [
    "hbl_status_string", "hbl_packed_weight_bytes", "hbl_workspace_bytes",
    "hbl_quantize_weights_workspace_bytes", "hbl_quantize_weights", "hbl_forward",
    "hbl_block_workspace_bytes", "hbl_block_forward", "hbl_check_status", "hbl_hadamard_f32", "hbl_hadamard_bf16", "hbl_forward_norm", "hbl_norm_quantize_act", "hbl_forward_glu", "hbl_glu_quantize_act", "hbl_quantize_weights_rotated", "hbl_quantize_weights_rotated_workspace_bytes",
    "hbl_quantize_act", "hbl_gemm_i32", "hbl_unpack_weights", "hbl_forward_host", "hbl_launch_count",
    "hbl_profile_events", "hbl_gemm_i32_static", "hbl_kv_codes_bytes", "hbl_quantize_kv",
    "hbl_selftest_wait_timeout", "hbl_quantize_act_int4_packed", "hbl_gemm_i32_int4_packed",
]

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhbl.so")
_lib = None


class HblError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class hbl_block_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("x_attn_in", "x_o_in", "x_ffn_in", "x_down_in",
                                          "Wq", "Wk", "Wv", "Wo", "Wup", "Wgate", "Wdown", "alpha7",
                                          "yq", "yk", "yv", "yo", "yup", "ygate", "ydown")] + \
               [("tokens", C.c_int), ("hidden", C.c_int), ("ffn", C.c_int), ("bits", C.c_int),
                ("x_dtype", C.c_int), ("eps", C.c_float)]


def lib() -> C.CDLL:
    """Loads libhbl.so (built by paper_2504_18415_b200.build).  Raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2504_18415_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.hbl_status_string.restype = C.c_char_p
        L.hbl_status_string.argtypes = [C.c_int]
        for n in ("hbl_packed_weight_bytes", "hbl_quantize_weights_workspace_bytes",
                  "hbl_quantize_weights_rotated_workspace_bytes"):
            getattr(L, n).restype = C.c_size_t
            getattr(L, n).argtypes = [C.c_int, C.c_int]
        for n in ("hbl_workspace_bytes", "hbl_block_workspace_bytes"):
            getattr(L, n).restype = C.c_size_t
            getattr(L, n).argtypes = [C.c_int, C.c_int, C.c_int]
        vp, i, f, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
        L.hbl_quantize_weights.argtypes = [vp, i, i, i, f, vp, vp, vp, sz, vp]
        L.hbl_quantize_weights_rotated.argtypes = [vp, i, i, i, f, vp, vp, vp, sz, vp]
        L.hbl_quantize_weights_rotated.restype = C.c_int
        L.hbl_forward.argtypes = [vp, i, i, i, vp, vp, i, i, i, f, vp, vp, sz, i, vp]
        L.hbl_block_forward.argtypes = [C.POINTER(hbl_block_t), vp, sz, i, vp]
        L.hbl_check_status.argtypes = [vp]
        L.hbl_hadamard_f32.argtypes = [vp, i, i, i, vp, vp]
        L.hbl_hadamard_bf16.argtypes = [vp, i, i, vp, vp]
        L.hbl_forward_norm.argtypes = [vp, vp, i, f, i, i, vp, vp, i, i, f, vp, vp, sz, i, vp]
        L.hbl_norm_quantize_act.argtypes = [vp, vp, i, f, i, i, i, f, vp, vp, vp, vp, vp]
        L.hbl_forward_glu.argtypes = [vp, vp, i, i, vp, vp, i, i, f, vp, vp, sz, i, vp]
        L.hbl_glu_quantize_act.argtypes = [vp, vp, i, i, i, f, vp, vp, vp, vp, vp]
        L.hbl_quantize_act.argtypes = [vp, i, i, i, i, i, f, vp, vp, vp, vp]
        L.hbl_gemm_i32.argtypes = [vp, vp, i, i, vp, i, vp, vp, sz, i, vp]
        L.hbl_unpack_weights.argtypes = [vp, i, i, vp, vp]
        L.hbl_gemm_i32_static.argtypes = [vp, vp, i, i, vp, i, vp, vp]
        L.hbl_gemm_i32_static.restype = C.c_int
        L.hbl_kv_codes_bytes.restype = C.c_size_t
        L.hbl_kv_codes_bytes.argtypes = [i, i, i, i]
        L.hbl_quantize_kv.restype = C.c_int
        L.hbl_quantize_kv.argtypes = [vp, i, i, i, i, i, f, vp, vp, vp, vp, vp]
        L.hbl_quantize_act_int4_packed.restype = C.c_int
        L.hbl_quantize_act_int4_packed.argtypes = [vp, i, i, i, i, f, vp, vp, vp]
        L.hbl_gemm_i32_int4_packed.restype = C.c_int
        L.hbl_gemm_i32_int4_packed.argtypes = [vp, i, i, vp, i, vp, vp, sz, vp]
        L.hbl_selftest_wait_timeout.restype = C.c_int
        L.hbl_selftest_wait_timeout.argtypes = [i, vp, vp]
        L.hbl_forward_host.argtypes = [vp, i, i, i, vp, vp, i, i, i, f, vp, vp, vp, vp, sz, i, vp]
        L.hbl_forward_host.restype = C.c_int
        L.hbl_launch_count.restype = C.c_ulonglong
        L.hbl_launch_count.argtypes = []
        L.hbl_profile_events.argtypes = [C.POINTER(vp), C.POINTER(vp), i, i]
        L.hbl_profile_events.restype = C.c_int
        for n in ("hbl_quantize_weights", "hbl_forward", "hbl_block_forward", "hbl_check_status",
                  "hbl_hadamard_f32", "hbl_hadamard_bf16", "hbl_forward_norm", "hbl_norm_quantize_act", "hbl_forward_glu", "hbl_glu_quantize_act", "hbl_quantize_act", "hbl_gemm_i32", "hbl_unpack_weights"):
            getattr(L, n).restype = C.c_int
        _lib = L
    return _lib


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return HBL_F32
    if t.dtype == torch.bfloat16:
        return HBL_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, where: str):
    if rc != HBL_OK:
        raise HblError(rc, where)


def hbl_packed_weight_bytes(out_dim: int, in_dim: int) -> int:
    return int(lib().hbl_packed_weight_bytes(out_dim, in_dim))


def hbl_workspace_bytes(max_tokens: int, in_dim: int, out_dim: int) -> int:
    return int(lib().hbl_workspace_bytes(max_tokens, in_dim, out_dim))


def hbl_block_workspace_bytes(max_tokens: int, hidden: int, ffn: int) -> int:
    return int(lib().hbl_block_workspace_bytes(max_tokens, hidden, ffn))


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 1024-byte aligned uint8 scratch tensor (torch's allocator aligns to 512 B; over-allocate)."""
    raw = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
    off = (-raw.data_ptr()) % 1024
    return raw[off:off + nbytes]


def hbl_quantize_weights(W_latent: torch.Tensor, eps: float = 1e-5):
    """Eq. 1-2.  Returns (W_packed uint8 tensor, alpha fp32 tensor of one element), both on device."""
    N, K = W_latent.shape
    nbytes = hbl_packed_weight_bytes(N, K)
    if nbytes == 0:
        raise HblError(2, "hbl_quantize_weights")
    packed = torch.empty(nbytes, dtype=torch.uint8, device=W_latent.device)
    alpha = torch.empty(1, dtype=torch.float32, device=W_latent.device)
    ws_bytes = int(lib().hbl_quantize_weights_workspace_bytes(N, K))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=W_latent.device)
    _check(lib().hbl_quantize_weights(_ptr(W_latent), _dt(W_latent), N, K, eps, _ptr(packed), _ptr(alpha),
                                      _ptr(ws), ws_bytes, _stream()), "hbl_quantize_weights")
    return packed, alpha


def hbl_quantize_weights_rotated(W_latent: torch.Tensor, eps: float = 1e-5):
    """Ternarises W H (each row transformed first): the weight-and-activation-rotation variant.  Returns as
    hbl_quantize_weights."""
    N, K = W_latent.shape
    nbytes = hbl_packed_weight_bytes(N, K)
    if nbytes == 0:
        raise HblError(2, "hbl_quantize_weights_rotated")
    packed = torch.empty(nbytes, dtype=torch.uint8, device=W_latent.device)
    alpha = torch.empty(1, dtype=torch.float32, device=W_latent.device)
    ws_bytes = int(lib().hbl_quantize_weights_rotated_workspace_bytes(N, K))
    ws = new_workspace(ws_bytes, W_latent.device)
    _check(lib().hbl_quantize_weights_rotated(_ptr(W_latent), _dt(W_latent), N, K, eps, _ptr(packed), _ptr(alpha),
                                              _ptr(ws), ws.numel(), _stream()), "hbl_quantize_weights_rotated")
    return packed, alpha


def hbl_forward(x: torch.Tensor, W_packed: torch.Tensor, alpha: torch.Tensor, out_dim: int, bits: int,
                use_hadamard: bool, eps: float = 1e-5, y: torch.Tensor | None = None,
                workspace: torch.Tensor | None = None, path: int = PATH_AUTO) -> torch.Tensor:
    """Eq. 3-7.  x [T,K] fp32/bf16 -> y [T,N] bf16."""
    T, K = x.shape
    if y is None:
        y = torch.empty((T, out_dim), dtype=torch.bfloat16, device=x.device)
    if workspace is None:
        workspace = new_workspace(hbl_workspace_bytes(T, K, out_dim), x.device)
    _check(lib().hbl_forward(_ptr(x), _dt(x), T, K, _ptr(W_packed), _ptr(alpha), out_dim, bits,
                             int(bool(use_hadamard)), eps, _ptr(y), _ptr(workspace), workspace.numel(),
                             path, _stream()), "hbl_forward")
    return y


def hbl_block_forward(inputs: dict, weights: dict, alpha7: torch.Tensor, hidden: int, ffn: int, bits: int,
                      eps: float = 1e-5, outputs: dict | None = None, workspace: torch.Tensor | None = None,
                      path: int = PATH_AUTO) -> dict:
    """The seven projections of one decoder block.  inputs: attn_in, o_in, ffn_in, down_in;
    weights (packed): q,k,v,o,up,gate,down; alpha7 in that order.  Returns the seven bf16 outputs."""
    T = inputs["attn_in"].shape[0]
    dev = inputs["attn_in"].device
    dims = {"q": hidden, "k": hidden, "v": hidden, "o": hidden, "up": ffn, "gate": ffn, "down": hidden}
    if outputs is None:
        outputs = {n: torch.empty((T, d), dtype=torch.bfloat16, device=dev) for n, d in dims.items()}
    if workspace is None:
        workspace = new_workspace(hbl_block_workspace_bytes(T, hidden, ffn), dev)
    b = hbl_block_t()
    for n in ("attn_in", "o_in", "ffn_in", "down_in"):
        t = inputs.get(n)                                    # no "down_in": the call chains SiLU(gate) * up into W_down
        setattr(b, "x_" + n, t.data_ptr() if t is not None else None)
    for n in dims:
        setattr(b, "W" + n, weights[n].data_ptr())
        setattr(b, "y" + n, outputs[n].data_ptr())
    b.alpha7 = alpha7.data_ptr()
    b.tokens, b.hidden, b.ffn, b.bits = T, hidden, ffn, bits
    b.x_dtype, b.eps = _dt(inputs["attn_in"]), eps
    _check(lib().hbl_block_forward(C.byref(b), _ptr(workspace), workspace.numel(), path, _stream()),
           "hbl_block_forward")
    return outputs


def hbl_check_status() -> int:
    return int(lib().hbl_check_status(_stream()))


def hbl_hadamard_f32(x: torch.Tensor) -> torch.Tensor:
    T, K = x.shape
    out = torch.empty((T, K), dtype=torch.float32, device=x.device)
    _check(lib().hbl_hadamard_f32(_ptr(x), _dt(x), T, K, _ptr(out), _stream()), "hbl_hadamard_f32")
    return out


def hbl_hadamard_bf16(g: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """bf16 [T,K] -> bf16 [T,K]: the orthonormal transform alone (the backward pass applies it to the gradient)."""
    T, K = g.shape
    if out is None:
        out = torch.empty((T, K), dtype=torch.bfloat16, device=g.device)
    _check(lib().hbl_hadamard_bf16(_ptr(g), T, K, _ptr(out), _stream()), "hbl_hadamard_bf16")
    return out


def hbl_forward_norm(x: torch.Tensor, gain: torch.Tensor, norm_eps: float, W_packed: torch.Tensor, alpha: torch.Tensor,
                     out_dim: int, bits: int, eps: float = 1e-5, y: torch.Tensor | None = None,
                     workspace: torch.Tensor | None = None, path: int = PATH_AUTO) -> torch.Tensor:
    """hbl_forward with RMS normalisation and a gain vector fused in front of the transform (bf16 x; fp32 or bf16 gain)."""
    T, K = x.shape
    if y is None:
        y = torch.empty((T, out_dim), dtype=torch.bfloat16, device=x.device)
    if workspace is None:
        workspace = new_workspace(hbl_workspace_bytes(T, K, out_dim), x.device)
    _check(lib().hbl_forward_norm(_ptr(x), _ptr(gain), _dt(gain), norm_eps, T, K, _ptr(W_packed), _ptr(alpha), out_dim, bits, eps,
                                  _ptr(y), _ptr(workspace), workspace.numel(), path, _stream()), "hbl_forward_norm")
    return y


def hbl_forward_glu(gate: torch.Tensor, up: torch.Tensor, W_packed: torch.Tensor, alpha: torch.Tensor, out_dim: int,
                    bits: int, eps: float = 1e-5, y: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                    path: int = PATH_AUTO) -> torch.Tensor:
    """The down projection with SiLU(gate) * up fused in front of the transform (bf16 gate and up)."""
    T, K = gate.shape
    if y is None:
        y = torch.empty((T, out_dim), dtype=torch.bfloat16, device=gate.device)
    if workspace is None:
        workspace = new_workspace(hbl_workspace_bytes(T, K, out_dim), gate.device)
    _check(lib().hbl_forward_glu(_ptr(gate), _ptr(up), T, K, _ptr(W_packed), _ptr(alpha), out_dim, bits, eps, _ptr(y),
                                 _ptr(workspace), workspace.numel(), path, _stream()), "hbl_forward_glu")
    return y


def hbl_glu_quantize_act(gate: torch.Tensor, up: torch.Tensor, bits: int, eps: float = 1e-5, export_xr: bool = False):
    """Gating product, transform, quantize.  Returns (codes, scale, codesum), or the fp32 H x' when export_xr."""
    T, K = gate.shape
    if export_xr:
        xr = torch.empty((T, K), dtype=torch.float32, device=gate.device)
        _check(lib().hbl_glu_quantize_act(_ptr(gate), _ptr(up), T, K, bits, eps, None, None, None, _ptr(xr), _stream()),
               "hbl_glu_quantize_act")
        return xr
    codes = torch.empty((T, K), dtype=torch.int8, device=gate.device)
    scale = torch.empty((T,), dtype=torch.float32, device=gate.device)
    csum = torch.empty((T,), dtype=torch.int32, device=gate.device)
    _check(lib().hbl_glu_quantize_act(_ptr(gate), _ptr(up), T, K, bits, eps, _ptr(codes), _ptr(scale), _ptr(csum), None,
                                      _stream()), "hbl_glu_quantize_act")
    return codes, scale, csum


def hbl_norm_quantize_act(x: torch.Tensor, gain: torch.Tensor, norm_eps: float, bits: int, eps: float = 1e-5,
                          export_xr: bool = False):
    """Normalise, transform, quantize.  Returns (codes, scale, codesum), or the fp32 H x' when export_xr."""
    T, K = x.shape
    if export_xr:
        xr = torch.empty((T, K), dtype=torch.float32, device=x.device)
        _check(lib().hbl_norm_quantize_act(_ptr(x), _ptr(gain), _dt(gain), norm_eps, T, K, bits, eps, None, None, None, _ptr(xr),
                                           _stream()), "hbl_norm_quantize_act")
        return xr
    codes = torch.empty((T, K), dtype=torch.int8, device=x.device)
    scale = torch.empty((T,), dtype=torch.float32, device=x.device)
    csum = torch.empty((T,), dtype=torch.int32, device=x.device)
    _check(lib().hbl_norm_quantize_act(_ptr(x), _ptr(gain), _dt(gain), norm_eps, T, K, bits, eps, _ptr(codes), _ptr(scale),
                                       _ptr(csum), None, _stream()), "hbl_norm_quantize_act")
    return codes, scale, csum


def hbl_quantize_act(x: torch.Tensor, bits: int, use_hadamard: bool, eps: float = 1e-5):
    """Returns (codes int8 [T,K], scale fp32 [T], codesum int32 [T])."""
    T, K = x.shape
    codes = torch.empty((T, K), dtype=torch.int8, device=x.device)
    scale = torch.empty((T,), dtype=torch.float32, device=x.device)
    csum = torch.empty((T,), dtype=torch.int32, device=x.device)
    _check(lib().hbl_quantize_act(_ptr(x), _dt(x), T, K, bits, int(bool(use_hadamard)), eps, _ptr(codes),
                                  _ptr(scale), _ptr(csum), _stream()), "hbl_quantize_act")
    return codes, scale, csum


def hbl_quantize_act_int4_packed(x: torch.Tensor, use_hadamard: bool, eps: float = 1e-5):
    """Eq. 3-4, 6 with the pack step: returns (codes uint8 [T, K/2], two INT4 codes per byte, scale fp32 [T])."""
    T, K = x.shape
    codes = torch.empty((T, K // 2), dtype=torch.uint8, device=x.device)
    scale = torch.empty((T,), dtype=torch.float32, device=x.device)
    _check(lib().hbl_quantize_act_int4_packed(_ptr(x), _dt(x), T, K, int(bool(use_hadamard)), eps, _ptr(codes), _ptr(scale),
                                              _stream()), "hbl_quantize_act_int4_packed")
    return codes, scale


def hbl_gemm_i32_int4_packed(codes_packed: torch.Tensor, W_packed: torch.Tensor, out_dim: int,
                             workspace: torch.Tensor | None = None) -> torch.Tensor:
    T, K = codes_packed.shape[0], codes_packed.shape[1] * 2
    acc = torch.empty((T, out_dim), dtype=torch.int32, device=codes_packed.device)
    if workspace is None:
        workspace = new_workspace(hbl_workspace_bytes(T, K, out_dim), codes_packed.device)
    _check(lib().hbl_gemm_i32_int4_packed(_ptr(codes_packed), T, K, _ptr(W_packed), out_dim, _ptr(acc), _ptr(workspace),
                                          workspace.numel(), _stream()), "hbl_gemm_i32_int4_packed")
    return acc


def hbl_gemm_i32(codes: torch.Tensor, codesum: torch.Tensor | None, W_packed: torch.Tensor, out_dim: int,
                 path: int = PATH_AUTO, workspace: torch.Tensor | None = None) -> torch.Tensor:
    T, K = codes.shape
    acc = torch.empty((T, out_dim), dtype=torch.int32, device=codes.device)
    if workspace is None:
        workspace = new_workspace(hbl_workspace_bytes(T, K, out_dim), codes.device)
    _check(lib().hbl_gemm_i32(_ptr(codes), _ptr(codesum), T, K, _ptr(W_packed), out_dim, _ptr(acc),
                              _ptr(workspace), workspace.numel(), path, _stream()), "hbl_gemm_i32")
    return acc


def hbl_gemm_i32_static(codes: torch.Tensor, codesum: torch.Tensor, W_packed: torch.Tensor, out_dim: int) -> torch.Tensor:
    """hbl_gemm_i32 (streaming kernel) without a workspace argument: for hosts that cannot allocate
    or lend scratch memory, the scratch is a fixed array inside the library (see include/hbl.h for
    the size limits).  Only the result tensor is created here, by torch, as for every other call."""
    T, K = codes.shape
    acc = torch.empty((T, out_dim), dtype=torch.int32, device=codes.device)
    _check(lib().hbl_gemm_i32_static(_ptr(codes), _ptr(codesum), T, K, _ptr(W_packed), out_dim, _ptr(acc),
                                     _stream()), "hbl_gemm_i32_static")
    return acc


def hbl_quantize_kv(x: torch.Tensor, bits: int, seq_len: int = 0, eps: float = 1e-5):
    """Section 3.1: x bf16 [tokens, n_heads, head_dim] -> (packed codes uint8 [tokens*n_heads, head_dim*bits/8],
    scale fp32 [tokens*n_heads], bos_codes uint8 [n_seq, n_heads, head_dim] or None, bos_scale or None)."""
    T, H, D = x.shape
    nbytes = int(lib().hbl_kv_codes_bytes(T, H, D, bits))
    if nbytes == 0 and T > 0:
        raise HblError(2, "hbl_quantize_kv")
    codes = torch.empty((T * H, D * bits // 8), dtype=torch.uint8, device=x.device)
    scale = torch.empty((T * H,), dtype=torch.float32, device=x.device)
    bos_codes = bos_scale = None
    if seq_len > 0:
        n_seq = (T + seq_len - 1) // seq_len
        bos_codes = torch.empty((n_seq, H, D), dtype=torch.uint8, device=x.device)
        bos_scale = torch.empty((n_seq * H,), dtype=torch.float32, device=x.device)
    _check(lib().hbl_quantize_kv(_ptr(x), T, H, D, bits, seq_len, eps, _ptr(codes), _ptr(scale), _ptr(bos_codes),
                                 _ptr(bos_scale), _stream()), "hbl_quantize_kv")
    return codes, scale, bos_codes, bos_scale


def hbl_unpack_weights(W_packed: torch.Tensor, out_dim: int, in_dim: int) -> torch.Tensor:
    out = torch.empty((out_dim, in_dim), dtype=torch.int8, device=W_packed.device)
    _check(lib().hbl_unpack_weights(_ptr(W_packed), out_dim, in_dim, _ptr(out), _stream()), "hbl_unpack_weights")
    return out


def hbl_forward_host(x_host: torch.Tensor, W_packed: torch.Tensor, alpha: torch.Tensor, out_dim: int,
                     bits: int, use_hadamard: bool, y_host: torch.Tensor, x_stage: torch.Tensor,
                     y_stage: torch.Tensor, workspace: torch.Tensor, eps: float = 1e-5,
                     path: int = PATH_AUTO) -> torch.Tensor:
    """hbl_forward with host-resident (pinned) x and y; copies are enqueued on the current stream."""
    T, K = x_host.shape
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("x_host / y_host must be host tensors")
    _check(lib().hbl_forward_host(C.c_void_p(x_host.data_ptr()), _dt(x_host), T, K, _ptr(W_packed), _ptr(alpha),
                                  out_dim, bits, int(bool(use_hadamard)), eps, C.c_void_p(y_host.data_ptr()),
                                  _ptr(x_stage), _ptr(y_stage), _ptr(workspace), workspace.numel(), path,
                                  _stream()), "hbl_forward_host")
    return y_host


def hbl_selftest_wait_timeout(limit_us: int = 1000) -> torch.Tensor:
    """Launches the kernel whose bounded wait runs out (see include/hbl.h); returns the device int that the
    second waiting role sets when it leaves because of the abort flag.  hbl_check_status() then reports the timeout."""
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib().hbl_selftest_wait_timeout(limit_us, _ptr(flag), _stream()), "hbl_selftest_wait_timeout")
    return flag


def hbl_launch_count() -> int:
    return int(lib().hbl_launch_count())


class KernelTimer:
    """Brackets the next n launches of one kernel class (1 = activation, 2 = contraction, 3 = unpack)
    with CUDA events recorded by the library on the launching stream."""

    def __init__(self, n: int, kernel: int):
        self.n, self.kernel = n, kernel
        self.starts = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        self.stops = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        for e in self.starts + self.stops:      # torch creates the handle lazily, on first record
            e.record()
        self._a = (C.c_void_p * n)(*[e.cuda_event for e in self.starts])
        self._b = (C.c_void_p * n)(*[e.cuda_event for e in self.stops])
        self.used = 0

    def __enter__(self):
        rc = lib().hbl_profile_events(self._a, self._b, self.n, self.kernel)
        if rc < 0:
            raise HblError(-rc, "hbl_profile_events")
        return self

    def __exit__(self, *exc):
        self.used = lib().hbl_profile_events(None, None, 0, self.kernel)

    def times_ms(self):
        torch.cuda.synchronize()
        return [self.starts[i].elapsed_time(self.stops[i]) for i in range(self.used)]
