"""A bounded device-side wait that is seen to run out.

Every wait inside the pipelined kernels has a time limit, after which the kernel records HBL_ERR_TIMEOUT, its
roles leave their waits, and it returns normally.  The self-test kernel takes exactly that path (its barrier is
never arrived at); afterwards the status must read HBL_ERR_TIMEOUT once, then clean, and the library must work."""
import time

import numpy as np
import pytest
import torch

from paper_2504_18415_b200 import hbl, workloads as wl
from parity_utils import EPS, check_y, oracle_layer, to_dev

pytestmark = pytest.mark.gpu


def test_wait_runs_out_and_the_library_carries_on():
    assert hbl.hbl_check_status() == 0
    t0 = time.perf_counter()
    flag = hbl.hbl_selftest_wait_timeout(1000)                 # 1 ms limit
    st = hbl.hbl_check_status()                                # synchronises the stream
    dt = time.perf_counter() - t0
    assert st == 9, hbl.STATUS_NAMES.get(st, st)               # HBL_ERR_TIMEOUT
    assert flag.item() == 1                                    # the second role left through the abort flag ...
    assert dt < 1.0                                            # ... not through its own 2 s limit
    assert hbl.hbl_check_status() == 0                         # reported once, then cleared
    # both contraction kernels (tensor memory was freed) still give the oracle's results
    K, N, T = 1024, 784, 200
    x = wl.rows("attn_out", 21, 1, K, 0, T, "bf16")
    W = wl.rows("latent", 21, 2, K, 0, N, "f32")
    o = oracle_layer(x, W, 4, True)
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(W).cuda(), EPS)
    for path, rows in ((hbl.PATH_TENSOR, T), (hbl.PATH_STREAM, 100), (hbl.PATH_STREAM_OVERLAP, 100)):
        y = hbl.hbl_forward(to_dev(x[:rows], "bf16"), packed, alpha, N, 4, True, EPS, path=path)
        assert hbl.hbl_check_status() == 0
        check_y(y, o["y64"][:rows])


def test_selftest_argument_errors():
    L = hbl.lib()
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert L.hbl_selftest_wait_timeout(0, flag.data_ptr(), None) == 2
    assert L.hbl_selftest_wait_timeout(2000000, flag.data_ptr(), None) == 2
    assert L.hbl_selftest_wait_timeout(100, None, None) == 1
