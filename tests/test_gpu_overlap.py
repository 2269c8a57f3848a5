"""HBL_PATH_STREAM_OVERLAP: calls issued back to back whose quantizer runs beside the previous call's contraction.

The mode changes no arithmetic -- the same kernels on the same operands -- so every call must give, bit for bit,
what HBL_PATH_STREAM gives on the same inputs.  What it changes is what runs at the same time: the next call's
quantizer writes one half of the scratch while the previous contraction still reads the other, and an ordinary
call that follows must be held back until everything before it is complete.  The tests therefore issue long runs
of calls without a synchronisation in between, with inputs that change from call to call (a stale or overwritten
half shows as the wrong call's result), mix the modes on one workspace, and check that no bounded wait ran out."""
import pytest
import torch

from paper_2504_18415_b200 import hbl, workloads as wl

pytestmark = pytest.mark.gpu
EPS = 1e-5


def _weights(shapes, g):
    packed, alphas = {}, []
    for n, (N, K) in shapes.items():
        p, a = hbl.hbl_quantize_weights(torch.randn((N, K), device="cuda", generator=g) * 0.02, EPS)
        packed[n] = p
        alphas.append(a)
    return packed, torch.cat(alphas)


@pytest.mark.parametrize("T", [1, 16, 40, 130])
def test_block_back_to_back_calls_equal_plain_streaming_calls(T):
    cfg = wl.CONFIG5
    H, F = cfg.hidden, cfg.ffn
    g = torch.Generator(device="cuda").manual_seed(900 + T)
    packed, alpha7 = _weights(cfg.weight_shapes(), g)
    n_sets = 5                                     # odd: a set meets both halves of the scratch
    ins = [{"attn_in": torch.randn((T, H), device="cuda", generator=g).bfloat16(),
            "o_in": torch.randn((T, H), device="cuda", generator=g).bfloat16(),
            "ffn_in": torch.randn((T, H), device="cuda", generator=g).bfloat16(),
            "down_in": torch.randn((T, F), device="cuda", generator=g).abs().bfloat16()} for _ in range(n_sets)]
    work = hbl.new_workspace(hbl.hbl_block_workspace_bytes(T, H, F))
    ref = []
    for i in range(n_sets):
        r = hbl.hbl_block_forward(ins[i], packed, alpha7, H, F, 4, EPS, workspace=work, path=hbl.PATH_STREAM)
        ref.append({n: v.clone() for n, v in r.items()})
    assert hbl.hbl_check_status() == 0
    outs = [{n: torch.empty_like(v) for n, v in ref[0].items()} for _ in range(n_sets)]
    for rep in range(40):
        for i in range(n_sets):                    # no synchronisation anywhere in here
            hbl.hbl_block_forward(ins[i], packed, alpha7, H, F, 4, EPS, outputs=outs[i], workspace=work,
                                  path=hbl.PATH_STREAM_OVERLAP)
        if rep % 10 == 9 or rep == 0:
            assert hbl.hbl_check_status() == 0, f"bounded wait ran out in round {rep}"
            for i in range(n_sets):
                for n in ref[i]:
                    assert torch.equal(outs[i][n], ref[i][n]), f"round {rep}, input set {i}, output {n} differs"


def test_block_modes_mixed_on_one_workspace():
    """An ordinary call directly after back-to-back calls (and the other way round) on the same workspace: the
    ordinary call must wait for the contraction before it, which released its dependents early."""
    cfg = wl.CONFIG5
    H, F, T = cfg.hidden, cfg.ffn, 16
    g = torch.Generator(device="cuda").manual_seed(77)
    packed, alpha7 = _weights(cfg.weight_shapes(), g)
    ins = [{"attn_in": torch.randn((T, H), device="cuda", generator=g).bfloat16(),
            "o_in": torch.randn((T, H), device="cuda", generator=g).bfloat16(),
            "ffn_in": torch.randn((T, H), device="cuda", generator=g).bfloat16(),
            "down_in": torch.randn((T, F), device="cuda", generator=g).abs().bfloat16()} for _ in range(3)]
    work = hbl.new_workspace(hbl.hbl_block_workspace_bytes(T, H, F))
    ref = []
    for i in range(3):
        r = hbl.hbl_block_forward(ins[i], packed, alpha7, H, F, 4, EPS, workspace=work, path=hbl.PATH_TENSOR)
        ref.append({n: v.clone() for n, v in r.items()})
    outs = [{n: torch.empty_like(v) for n, v in ref[0].items()} for _ in range(3)]
    modes = [hbl.PATH_STREAM_OVERLAP, hbl.PATH_STREAM_OVERLAP, hbl.PATH_STREAM, hbl.PATH_STREAM_OVERLAP, hbl.PATH_AUTO,
             hbl.PATH_STREAM_OVERLAP, hbl.PATH_TENSOR, hbl.PATH_STREAM_OVERLAP, hbl.PATH_STREAM_OVERLAP]
    for rep in range(30):
        for k, m in enumerate(modes):
            i = (rep + k) % 3
            hbl.hbl_block_forward(ins[i], packed, alpha7, H, F, 4, EPS, outputs=outs[i], workspace=work, path=m)
            if rep % 10 == 0:
                # checked call by call here (the comparison synchronises), in full flight in the other rounds
                for n in ref[i]:
                    assert torch.equal(outs[i][n], ref[i][n]), f"round {rep}, call {k} (mode {m}), output {n} differs"
    assert hbl.hbl_check_status() == 0
    for i in range(3):                             # after the rounds in full flight: every set was last written by some mode
        for n in ref[i]:
            assert torch.equal(outs[i][n], ref[i][n]), f"input set {i}, output {n} differs after the last round"


@pytest.mark.parametrize("cfg,T", [(wl.CONFIG4B, 16), (wl.CONFIG3, 16), (wl.CONFIG2, 1), (wl.CONFIG4A, 150)],
                         ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_layer_back_to_back_calls_equal_plain_streaming_calls(cfg, T):
    g = torch.Generator(device="cuda").manual_seed(5 + T)
    W = torch.randn((cfg.N, cfg.K), device="cuda", generator=g) * 0.02
    packed, alpha = hbl.hbl_quantize_weights(W, EPS)
    xs = [torch.randn((T, cfg.K), device="cuda", generator=g).bfloat16() for _ in range(3)]
    work = hbl.new_workspace(hbl.hbl_workspace_bytes(T, cfg.K, cfg.N))
    ref = [hbl.hbl_forward(x, packed, alpha, cfg.N, cfg.bits, cfg.use_hadamard, EPS, workspace=work,
                           path=hbl.PATH_STREAM).clone() for x in xs]
    ys = [torch.empty_like(r) for r in ref]
    for rep in range(60):
        for i in range(3):
            hbl.hbl_forward(xs[i], packed, alpha, cfg.N, cfg.bits, cfg.use_hadamard, EPS, y=ys[i], workspace=work,
                            path=hbl.PATH_STREAM_OVERLAP)
    assert hbl.hbl_check_status() == 0
    for i in range(3):
        assert torch.equal(ys[i], ref[i]), f"input {i} differs"


@pytest.mark.parametrize("dtype,K,had", [(torch.float32, 4096, True), (torch.bfloat16, 1024, True), (torch.float32, 1536, False)])
def test_layer_back_to_back_without_the_counting_quantizer(dtype, K, had):
    """Inputs the one-launch quantizer does not serve (fp32, or a transform size outside 2^11..2^14): the mode then
    rests on the quantizer's completion alone.  Same bar: bit-equality with plain streaming calls."""
    N, T = 1024, 24
    g = torch.Generator(device="cuda").manual_seed(K + T)
    packed, alpha = hbl.hbl_quantize_weights(torch.randn((N, K), device="cuda", generator=g) * 0.02, EPS)
    xs = [torch.randn((T, K), device="cuda", generator=g).to(dtype) for _ in range(3)]
    work = hbl.new_workspace(hbl.hbl_workspace_bytes(T, K, N))
    ref = [hbl.hbl_forward(x, packed, alpha, N, 4, had, EPS, workspace=work, path=hbl.PATH_STREAM).clone() for x in xs]
    ys = [torch.empty_like(r) for r in ref]
    for rep in range(60):
        for i in range(3):
            hbl.hbl_forward(xs[i], packed, alpha, N, 4, had, EPS, y=ys[i], workspace=work, path=hbl.PATH_STREAM_OVERLAP)
    assert hbl.hbl_check_status() == 0
    for i in range(3):
        assert torch.equal(ys[i], ref[i]), f"input {i} differs"


def test_automatic_path_sees_chained_layers():
    """The automatic path takes the back-to-back mode by itself when the call's inputs are clear of what the call
    before it writes.  Here they are not: the second layer reads the first layer's output, directly, with nothing in
    between.  Runs of such pairs, inputs taking turns, must give what two synchronised large-batch calls give."""
    T, K, N1, N2 = 16, 4096, 4096, 2048
    g = torch.Generator(device="cuda").manual_seed(321)
    p1, a1 = hbl.hbl_quantize_weights(torch.randn((N1, K), device="cuda", generator=g) * 0.02, EPS)
    p2, a2 = hbl.hbl_quantize_weights(torch.randn((N2, N1), device="cuda", generator=g) * 0.02, EPS)
    xs = [torch.randn((T, K), device="cuda", generator=g).bfloat16() for _ in range(3)]
    ref = []
    for x in xs:
        y1 = hbl.hbl_forward(x, p1, a1, N1, 4, True, EPS, path=hbl.PATH_TENSOR)
        ref.append(hbl.hbl_forward(y1, p2, a2, N2, 4, True, EPS, path=hbl.PATH_TENSOR).clone())
    w1 = hbl.new_workspace(hbl.hbl_workspace_bytes(T, K, N1))
    w2 = hbl.new_workspace(hbl.hbl_workspace_bytes(T, N1, N2))
    y1 = torch.empty((T, N1), dtype=torch.bfloat16, device="cuda")
    y2 = [torch.empty((T, N2), dtype=torch.bfloat16, device="cuda") for _ in xs]
    for rep in range(60):
        for i, x in enumerate(xs):
            hbl.hbl_forward(x, p1, a1, N1, 4, True, EPS, y=y1, workspace=w1)          # automatic path
            hbl.hbl_forward(y1, p2, a2, N2, 4, True, EPS, y=y2[i], workspace=w2)      # reads what the call before wrote
    assert hbl.hbl_check_status() == 0
    for i in range(3):
        assert torch.equal(y2[i], ref[i]), f"input {i} differs"


def test_automatic_path_one_buffer_two_layouts():
    """One scratch buffer lent to calls of two token counts in turn: same base, different layouts, so the halves of
    one call are not the halves of the next.  The automatic path has to notice (it compares the whole workspace
    range with the one the call before used) and must not let the second call's quantizer write while the first
    call's contraction still reads."""
    cfg = wl.CONFIG4A
    N, K = cfg.N, cfg.K
    g = torch.Generator(device="cuda").manual_seed(99)
    packed, alpha = hbl.hbl_quantize_weights(torch.randn((N, K), device="cuda", generator=g) * 0.02, EPS)
    Ts = [16, 64, 5, 64, 16]
    xs = [torch.randn((T, K), device="cuda", generator=g).bfloat16() for T in Ts]
    ref = [hbl.hbl_forward(x, packed, alpha, N, cfg.bits, cfg.use_hadamard, EPS, path=hbl.PATH_TENSOR).clone() for x in xs]
    work = hbl.new_workspace(max(hbl.hbl_workspace_bytes(T, K, N) for T in Ts))
    ys = [torch.empty_like(r) for r in ref]
    for rep in range(60):
        for i, x in enumerate(xs):
            hbl.hbl_forward(x, packed, alpha, N, cfg.bits, cfg.use_hadamard, EPS, y=ys[i], workspace=work[:hbl.hbl_workspace_bytes(Ts[i], K, N)])
    assert hbl.hbl_check_status() == 0
    for i in range(len(xs)):
        assert torch.equal(ys[i], ref[i]), f"call {i} ({Ts[i]} tokens) differs"
