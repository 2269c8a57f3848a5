"""The workspace-free contraction entry point, hbl_gemm_i32_static.

Some hosts cannot allocate device memory when they call the library (all of it was
handed to a cache pool at start-up, or the call sits where an allocation would
synchronise the device), so this entry point keeps the streaming kernel's scratch
in a fixed array inside the library.  It must give exactly what hbl_gemm_i32 gives
on the streaming kernel -- integer work, so bit for bit -- and, because every call
shares that array and inherits the previous call's leftovers, it must do so on
calls made back to back, on shapes that leave different leftovers behind.

This file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import hbl_oracle as orc
from paper_2504_18415_b200 import hbl, workloads as wl

EPS = 1e-5


def _problem(T, K, N, bits, seed):
    rng = np.random.default_rng(seed)
    lo, hi = (-128, 128) if bits == 8 else (-8, 8)
    q = torch.from_numpy(rng.integers(lo, hi, size=(T, K), dtype=np.int8)).cuda()
    W = wl.rows("latent", seed, 60, K, 0, N, "f32")
    packed, _ = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    return q, q.to(torch.int32).sum(1, dtype=torch.int32), packed


@pytest.mark.gpu
def test_static_scratch_matches_workspace_version_on_consecutive_calls():
    # shapes whose row blocks are shared between thread blocks (scratch is really used), a ragged token
    # count, then a smaller problem that would trip over the first one's flags if they were not cleared
    shapes = [(16, 8192, 2048, 4), (5, 4096, 528, 8), (16, 8192, 2048, 4), (1, 2048, 2048, 4)]
    for n, (T, K, N, bits) in enumerate(shapes):
        q, csum, packed = _problem(T, K, N, bits, 700 + n)
        want = hbl.hbl_gemm_i32(q, csum, packed, N, hbl.PATH_STREAM)
        got = hbl.hbl_gemm_i32_static(q, csum, packed, N)
        again = hbl.hbl_gemm_i32_static(q, csum, packed, N)
        assert hbl.hbl_check_status() == 0
        assert torch.equal(got, want), f"call {n}: first static call differs"
        assert torch.equal(again, want), f"call {n}: second static call differs"
        # and both are the exact integer contraction, as the CPU oracle computes it
        wt = hbl.hbl_unpack_weights(packed, N, K).cpu().numpy()
        assert np.array_equal(got.cpu().numpy(), orc.gemm(q.cpu().numpy(), wt)), f"call {n}: differs from the oracle"


@pytest.mark.gpu
def test_static_scratch_zero_tokens():
    _, _, packed = _problem(1, 128, 16, 4, 3)
    out = hbl.hbl_gemm_i32_static(torch.empty((0, 128), dtype=torch.int8, device="cuda"),
                                  torch.empty((0,), dtype=torch.int32, device="cuda"), packed, 16)
    assert out.shape == (0, 16)


def test_sizes_beyond_the_fixed_array_are_refused_on_the_host():
    L = hbl.lib()
    p, n = C.c_void_p(1024), C.c_void_p(0)
    call = lambda T, K, N: L.hbl_gemm_i32_static(p, p, T, K, p, N, p, n)
    assert call(65, 1024, 1024) == 11          # the fixed array holds slots for 16 tokens
    assert call(64, 1024, 8192) == 11
    assert call(17, 1024, 1024) == 11
    assert call(16, 65536, 1024) == 11         # in_dim beyond the library's maximum
    assert call(16, 1000, 1024) == 2           # shape errors still come first
    assert call(0, 1024, 1024) == 0            # nothing to do
