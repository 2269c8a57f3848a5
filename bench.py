#!/usr/bin/env python
"""Benchmark of the H-BitLinear forward path (one JSON line on stdout).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--sweep none|quick|full]

A "step" is one hbl_forward call (transform + quantize + contraction + rescale)
over one batch of the headline workload: the W_down-shaped H-BitLinear layer of
the 1.3B model (in 8192 -> out 2048, INT4 activations, Hadamard on) at 16384
tokens.  `value` is tokens/s with inputs resident in HBM; `e2e` is the same
call fed from pinned host memory with the copies inside the timed region.
The other workload points (small-batch weight streaming, the INT8 setting, the
7B decoder block) are reported under "points".

With N > 1 (torchrun, one rank per GPU) every rank runs an independent replica
of the same step (tokens are independent: no collective on the data path); the
time is the max over ranks and `value` the sum of tokens over ranks.

`--impl reference` times the CPU oracle (the only reference implementation
there is) on a bounded token sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

EPS = 1e-5
L2_BYTES = 126 * 1024 * 1024
RING_BYTES = 4 * L2_BYTES            # ring of distinct input sets so that every call is L2-cold
NOMINAL_INT8_TOPS = 4500.0
NOMINAL_HBM_GBS = 7700.0
METRIC = "H-BitLinear tokens/s and TOPS vs INT8 tensor peak; HBM GB/s at small batch"
UNIT = "tokens/s"
ALU_PEAK_LANE_OPS = 148 * 128 * 1.965e9      # fp32 lanes x SMs x clocks.max.sm
# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel at the headline workload, copied
# from an ncu capture of that kernel (151.78 MB read + 48.57 MB written); a constant, not re-measured by a run.
# None whenever the kernel has changed since the counters were taken.
GEMM_TENSOR_TRAFFIC_BYTES = 200351744
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"]))}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            f = [c.strip() for c in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [c for c, p in zip(sm, power) if p > 0.5 * max(power)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def library_int8_peak(torch, sustain_s=1.5):
    """A library int8 GEMM (torch._int_mm, 8192^3) as a measured ceiling for the int8 tensor path: best of 10
    single calls (burst) and the mean rate of back-to-back calls over `sustain_s` seconds (under the power cap).
    A baseline only: nothing of the product runs through it.  Returns TOPS or None where the call is unavailable."""
    try:
        n = 8192
        g = torch.Generator(device="cuda").manual_seed(1)
        a = torch.randint(-8, 8, (n, n), device="cuda", dtype=torch.int8, generator=g)
        b = torch.randint(-1, 2, (n, n), device="cuda", dtype=torch.int8, generator=g).t()   # K-major second operand
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); torch._int_mm(a, b); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        ops = 2.0 * n ** 3
        reps = max(10, int(sustain_s * 1e3 / best))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch._int_mm(a, b)
        e1.record()
        torch.cuda.synchronize()
        sus = e0.elapsed_time(e1) / reps
        return {"int8_library_tops_burst": round(ops / (best * 1e-3) / 1e12, 1),
                "int8_library_tops_sustained": round(ops / (sus * 1e-3) / 1e12, 1),
                "int8_library": "torch._int_mm 8192^3, best of 10 / mean over %.1f s back to back" % sustain_s}
    except Exception as exc:                                    # noqa: BLE001 -- a missing library kernel is not an error here
        return {"int8_library_tops_burst": None, "int8_library_tops_sustained": None,
                "int8_library": f"unavailable: {type(exc).__name__}: {exc}"[:200]}


# ----------------------------------------------------------------------------- workload helpers
def alg_bytes(T, K, N, x_bytes=2):
    """Algorithmic HBM bytes of one layer call: activations in, packed weights, bf16 out."""
    return T * K * x_bytes + N * K // 4 + 2 * T * N + 4


def device_x(cfg_kind, seed, tid, K, T, dtype, torch, max_host_rows=4096):
    """Activations per the workload recipe; beyond max_host_rows the seeded block is tiled."""
    from paper_2504_18415_b200 import workloads as wl
    rows = min(T, max_host_rows)
    x = torch.from_numpy(wl.rows(cfg_kind, seed, tid, K, 0, rows, dtype)).cuda()
    if dtype == "bf16":
        x = x.to(torch.bfloat16)
    if rows < T:
        x = x.repeat((T + rows - 1) // rows, 1)[:T].contiguous()
    return x


def device_weights(N, K, seed, torch, hbl):
    """Latent N(0, 0.02^2) weights drawn on the device (seeded), ternarised by the library."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    W = torch.randn((N, K), generator=g, device="cuda", dtype=torch.float32) * 0.02
    packed, alpha = hbl.hbl_quantize_weights(W, EPS)
    del W
    return packed, alpha


def max_over_ranks(total_ms, dist, device):
    """Device time of the slowest rank (MAX all-reduce) followed by a barrier; identity without a group."""
    if dist is None:
        return float(total_ms)
    import torch
    t = torch.tensor([float(total_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.barrier()
    return float(t.item())


def whole_job_value(world, tokens_per_rank, ms_per_step):
    """tokens/s summed over `world` independent replicas that all ran the same step in ms_per_step."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def time_loop(fn, iters, warmup, torch):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def graph_ms(call, ring, reps, torch):
    """ms per call of `ring` back-to-back calls captured in one CUDA graph (launch latencies hide one another)."""
    for _ in range(2):
        for _ in range(ring):
            call()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(ring):
            call()
    return time_loop(g.replay, reps, 3, torch) / ring


def layer_point(name, kind, seed, K, N, bits, had, T, torch, hbl, peaks, iters=None):
    """One single-layer workload point, L2-cold (ring of distinct input sets), returns a dict."""
    per_call = alg_bytes(T, K, N) + T * K          # + the int8 codes round trip (implementation traffic)
    ring = max(2, min(64, -(-RING_BYTES // per_call)))
    if T * K * 2 > 2 * L2_BYTES:
        ring = 2
    xs, ws, ys = [], [], []
    x0 = device_x(kind, seed, 1, K, T, "bf16", torch)
    for r in range(ring):
        xs.append(torch.roll(x0, shifts=r, dims=0) if r else x0)
        ws.append(device_weights(N, K, 1000 * seed + r, torch, hbl))
        ys.append(torch.empty((T, N), dtype=torch.bfloat16, device="cuda"))
    wsb = hbl.hbl_workspace_bytes(T, K, N)
    work = hbl.new_workspace(wsb)
    state = {"i": 0, "path": hbl.PATH_AUTO}

    def call():
        r = state["i"] % ring
        state["i"] += 1
        hbl.hbl_forward(xs[r], ws[r][0], ws[r][1], N, bits, had, EPS, y=ys[r], workspace=work, path=state["path"])

    small = T <= 512                     # the streaming path: a few launches per call, timed as a CUDA graph
    ms_b2b = None
    if small:
        ms = graph_ms(call, ring, iters or 20, torch)
        # Where the automatic choice is the streaming kernel (the library's rule: up to 128 tokens, up to 192 with
        # 16 MiB or more of packed weights, up to 256 with 32 MiB or more), it runs these calls in its back-to-back
        # mode by itself: no input here is written by the call before it, which the library checks.  For comparison,
        # the same calls as ordinary launches, each starting when the call before it is complete.
        if T <= 128 or (T <= 192 and N * K // 4 >= 16 << 20) or (T <= 256 and N * K // 4 >= 32 << 20):
            state["i"], state["path"] = 0, hbl.PATH_STREAM
            ms_b2b = graph_ms(call, ring, iters or 20, torch)
    else:
        flops = 2.0 * T * K * N
        est_ms = max(0.02, flops / 2.0e15 * 1e3)
        n_it = iters or int(max(5, min(50, 200.0 / est_ms)))
        ms = time_loop(call, n_it, 3, torch)
    st = hbl.hbl_check_status()
    if st != 0:
        raise RuntimeError(f"device status {st} in {name}")
    tops = 2.0 * T * K * N / (ms * 1e-3) / 1e12
    gbs = alg_bytes(T, K, N) / (ms * 1e-3) / 1e9
    out = {"point": name, "tokens": T, "in": K, "out": N, "bits": bits, "hadamard": bool(had),
           "ms": round(ms, 5), "tokens_per_s": round(T / (ms * 1e-3), 1), "tops": round(tops, 2),
           "alg_gbs": round(gbs, 1), "ring": ring, "graph": small}
    if small or tops < 100:
        out["bound"] = "hbm"
        out["frac"] = round(gbs / peaks["hbm_gbs"], 4)
        out["frac_of_nominal_hbm"] = round(gbs / NOMINAL_HBM_GBS, 4)
        if ms_b2b is not None:
            out["ms_ordinary_launches"] = round(ms_b2b, 5)
            out["frac_ordinary_launches"] = round(alg_bytes(T, K, N) / (ms_b2b * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)
    else:
        out["bound"] = "tensor"
        out["frac"] = round(tops / (2 * peaks["bf16_tflops"]), 4)
        # calls of a millisecond and more run under the power cap: the sustained figure is their ceiling
        out["frac_of_sustained"] = round(tops / (2 * peaks["bf16_tflops_sustained"]), 4)
        out["frac_of_nominal_int8"] = round(tops / NOMINAL_INT8_TOPS, 4)
    del xs, ws, ys, work
    torch.cuda.empty_cache()
    return out


def backward_transform_point(K, T, torch, hbl, peaks, iters=None):
    """The transform's backward pass (the same orthonormal product on a bf16 gradient, bf16 out): bound by
    HBM, 4 B per element.  L2-cold: a ring of distinct gradient buffers larger than L2."""
    per_call = 4 * T * K
    ring = max(2, min(16, -(-RING_BYTES // per_call)))
    gen = torch.Generator(device="cuda").manual_seed(900 + K)
    gs = [torch.randn((T, K), device="cuda", generator=gen).bfloat16() for _ in range(ring)]
    outs = [torch.empty_like(g) for g in gs]
    state = {"i": 0}

    def call():
        r = state["i"] % ring
        state["i"] += 1
        hbl.hbl_hadamard_bf16(gs[r], outs[r])

    ms = time_loop(call, iters or 30, 3, torch)
    st = hbl.hbl_check_status()
    if st != 0:
        raise RuntimeError(f"device status {st} in backward transform K={K}")
    gbs = per_call / (ms * 1e-3) / 1e9
    out = {"point": "transform_backward_bf16", "tokens": T, "in": K, "out": K, "bits": 16, "hadamard": True,
           "ms": round(ms, 5), "tokens_per_s": round(T / (ms * 1e-3), 1), "tops": 0.0, "alg_gbs": round(gbs, 1),
           "ring": ring, "graph": False, "bound": "hbm", "frac": round(gbs / peaks["hbm_gbs"], 4),
           "frac_of_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4)}
    del gs, outs
    torch.cuda.empty_cache()
    return out


def weight_quantize_point(N, K, dtype_name, torch, hbl, peaks, iters=None):
    """Eq. 1-2 on one latent weight tensor: the absmean pass and the ternarise-and-pack pass each read the
    tensor once (it is larger than what stays in L2 between them, or nearly), 1/4 byte per weight written.
    L2-cold: a ring of distinct latent tensors larger than L2."""
    dt = torch.float32 if dtype_name == "f32" else torch.bfloat16
    esz = 4 if dtype_name == "f32" else 2
    per_call = 2 * N * K * esz + N * K // 4
    ring = max(2, min(8, -(-RING_BYTES // (N * K * esz))))
    gen = torch.Generator(device="cuda").manual_seed(300 + N + K)
    Ws = [(torch.randn((N, K), device="cuda", generator=gen) * 0.02).to(dt) for _ in range(ring)]
    packed = torch.empty(hbl.hbl_packed_weight_bytes(N, K), dtype=torch.uint8, device="cuda")
    alpha = torch.empty(1, dtype=torch.float32, device="cuda")
    L = hbl.lib()
    ws_bytes = int(L.hbl_quantize_weights_workspace_bytes(N, K))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    state = {"i": 0}

    def call():
        W = Ws[state["i"] % ring]
        state["i"] += 1
        rc = L.hbl_quantize_weights(W.data_ptr(), 0 if dtype_name == "f32" else 1, N, K, EPS, packed.data_ptr(),
                                    alpha.data_ptr(), ws.data_ptr(), ws_bytes, None)
        if rc != 0:
            raise RuntimeError(f"hbl_quantize_weights -> {rc}")

    ms = time_loop(call, iters or 30, 3, torch)
    gbs = per_call / (ms * 1e-3) / 1e9
    out = {"point": f"weight_quantize_{dtype_name}", "tokens": 0, "in": K, "out": N, "bits": 2, "hadamard": False,
           "ms": round(ms, 5), "weights_per_s": round(N * K / (ms * 1e-3), 1), "tops": 0.0, "alg_gbs": round(gbs, 1),
           "ring": ring, "graph": False, "bound": "hbm", "frac": round(gbs / peaks["hbm_gbs"], 4),
           "frac_of_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4)}
    del Ws
    torch.cuda.empty_cache()
    return out


def row_quantize_point(K, T, bits, torch, hbl, peaks, iters=None):
    """Eq. 5-6 on bf16 activations without the transform (the inputs of the plain BitLinear projections and of the
    INT8 configuration): 2 B read + 1 B written per element, L2-cold (ring of inputs larger than L2)."""
    per_call = 3 * T * K
    ring = max(2, min(16, -(-RING_BYTES // per_call)))
    gen = torch.Generator(device="cuda").manual_seed(500 + K + bits)
    xs = [torch.randn((T, K), device="cuda", generator=gen).bfloat16() for _ in range(ring)]
    codes = [torch.empty((T, K), dtype=torch.int8, device="cuda") for _ in range(ring)]
    scale = torch.empty((T,), dtype=torch.float32, device="cuda")
    csum = torch.empty((T,), dtype=torch.int32, device="cuda")
    L = hbl.lib()
    state = {"i": 0}

    def call():
        r = state["i"] % ring
        state["i"] += 1
        rc = L.hbl_quantize_act(xs[r].data_ptr(), 1, T, K, bits, 0, EPS, codes[r].data_ptr(), scale.data_ptr(),
                                csum.data_ptr(), None)
        if rc != 0:
            raise RuntimeError(f"hbl_quantize_act -> {rc}")

    ms = time_loop(call, iters or 30, 3, torch)
    gbs = per_call / (ms * 1e-3) / 1e9
    out = {"point": f"row_quantize_int{bits}", "tokens": T, "in": K, "out": K, "bits": bits, "hadamard": False,
           "ms": round(ms, 5), "tokens_per_s": round(T / (ms * 1e-3), 1), "tops": 0.0, "alg_gbs": round(gbs, 1),
           "ring": ring, "graph": False, "bound": "hbm", "frac": round(gbs / peaks["hbm_gbs"], 4),
           "frac_of_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4)}
    del xs, codes
    torch.cuda.empty_cache()
    return out


def kv_quantize_point(T, H, D, bits, torch, hbl, peaks, iters=None):
    """The low-bit attention-state quantizer (absmax per head, unsigned codes): 2 B read + bits/8 B written per
    element, L2-cold (ring of inputs larger than L2)."""
    per_call = T * H * D * 2 + T * H * D * bits // 8 + 4 * T * H
    ring = max(2, min(16, -(-RING_BYTES // per_call)))
    gen = torch.Generator(device="cuda").manual_seed(1000 + bits)
    xs = [torch.randn((T, H, D), device="cuda", generator=gen).bfloat16() for _ in range(ring)]
    codes = torch.empty((T * H, D * bits // 8), dtype=torch.uint8, device="cuda")
    scale = torch.empty((T * H,), dtype=torch.float32, device="cuda")
    L = hbl.lib()
    state = {"i": 0}

    def call():
        x = xs[state["i"] % ring]
        state["i"] += 1
        rc = L.hbl_quantize_kv(x.data_ptr(), T, H, D, bits, 0, EPS, codes.data_ptr(), scale.data_ptr(), None, None, None)
        if rc != 0:
            raise RuntimeError(f"hbl_quantize_kv -> {rc}")

    ms = time_loop(call, iters or 30, 3, torch)
    gbs = per_call / (ms * 1e-3) / 1e9
    out = {"point": f"kv_quantize_int{bits}", "tokens": T, "in": H * D, "out": H * D, "bits": bits, "hadamard": False,
           "ms": round(ms, 5), "tokens_per_s": round(T / (ms * 1e-3), 1), "tops": 0.0, "alg_gbs": round(gbs, 1),
           "ring": ring, "graph": False, "bound": "hbm", "frac": round(gbs / peaks["hbm_gbs"], 4),
           "frac_of_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4)}
    del xs
    torch.cuda.empty_cache()
    return out


def norm_quantize_point(K, T, torch, hbl, peaks, iters=None):
    """RMS normalisation + transform + INT4 quantizer in one kernel (the activation side of hbl_forward_norm):
    2 B read + 1 B written per element, L2-cold (ring of inputs larger than L2)."""
    per_call = 3 * T * K
    ring = max(2, min(16, -(-RING_BYTES // per_call)))
    gen = torch.Generator(device="cuda").manual_seed(700 + K)
    xs = [torch.randn((T, K), device="cuda", generator=gen).bfloat16() for _ in range(ring)]
    gain = (torch.rand((K,), device="cuda", generator=gen) + 0.5).bfloat16()     # bf16, as models store it
    codes = torch.empty((T, K), dtype=torch.int8, device="cuda")
    scale = torch.empty((T,), dtype=torch.float32, device="cuda")
    L = hbl.lib()
    state = {"i": 0}

    def call():
        x = xs[state["i"] % ring]
        state["i"] += 1
        rc = L.hbl_norm_quantize_act(x.data_ptr(), gain.data_ptr(), 1, 1e-5, T, K, 4, EPS, codes.data_ptr(), scale.data_ptr(),
                                     None, None, None)
        if rc != 0:
            raise RuntimeError(f"hbl_norm_quantize_act returned {rc}")

    ms = time_loop(call, iters or 30, 3, torch)
    gbs = per_call / (ms * 1e-3) / 1e9
    out = {"point": "norm_transform_quantize_int4", "tokens": T, "in": K, "out": K, "bits": 4, "hadamard": True,
           "ms": round(ms, 5), "tokens_per_s": round(T / (ms * 1e-3), 1), "tops": 0.0, "alg_gbs": round(gbs, 1),
           "ring": ring, "graph": False, "bound": "hbm", "frac": round(gbs / peaks["hbm_gbs"], 4),
           "frac_of_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4)}
    del xs
    torch.cuda.empty_cache()
    return out


def glu_quantize_point(K, T, torch, hbl, peaks, iters=None):
    """SiLU(gate) * up + transform + INT4 quantizer in one kernel (the activation side of hbl_forward_glu):
    2 x 2 B read + 1 B written per element, L2-cold."""
    per_call = 5 * T * K
    ring = max(2, min(16, -(-RING_BYTES // per_call)))
    gen = torch.Generator(device="cuda").manual_seed(800 + K)
    gs = [torch.randn((T, K), device="cuda", generator=gen).bfloat16() for _ in range(ring)]
    us = [torch.randn((T, K), device="cuda", generator=gen).bfloat16() for _ in range(ring)]
    codes = torch.empty((T, K), dtype=torch.int8, device="cuda")
    scale = torch.empty((T,), dtype=torch.float32, device="cuda")
    L = hbl.lib()
    state = {"i": 0}

    def call():
        r = state["i"] % ring
        state["i"] += 1
        rc = L.hbl_glu_quantize_act(gs[r].data_ptr(), us[r].data_ptr(), T, K, 4, EPS, codes.data_ptr(), scale.data_ptr(),
                                    None, None, None)
        if rc != 0:
            raise RuntimeError(f"hbl_glu_quantize_act returned {rc}")

    ms = time_loop(call, iters or 30, 3, torch)
    gbs = per_call / (ms * 1e-3) / 1e9
    out = {"point": "glu_transform_quantize_int4", "tokens": T, "in": K, "out": K, "bits": 4, "hadamard": True,
           "ms": round(ms, 5), "tokens_per_s": round(T / (ms * 1e-3), 1), "tops": 0.0, "alg_gbs": round(gbs, 1),
           "ring": ring, "graph": False, "bound": "hbm", "frac": round(gbs / peaks["hbm_gbs"], 4),
           "frac_of_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4)}
    del gs, us
    torch.cuda.empty_cache()
    return out


def block_point(T, torch, hbl, peaks, iters=None):
    """7B-shaped decoder-block projection sweep point (config 5)."""
    from paper_2504_18415_b200 import workloads as wl
    cfg = wl.CONFIG5
    H, F = cfg.hidden, cfg.ffn
    shapes = cfg.weight_shapes()
    w_bytes = sum(n * k // 4 for n, k in shapes.values())
    per_call = w_bytes + T * (3 * H + F) * 2 + 2 * T * (5 * H + 2 * F)
    small = T <= 512
    ring = max(2, min(8, -(-RING_BYTES // per_call))) if T < 4096 else 1
    ins = {"attn_in": device_x("gauss", cfg.seed, 10, H, T, "bf16", torch),
           "o_in": device_x("attn_out", cfg.seed, 11, H, T, "bf16", torch),
           "ffn_in": device_x("gauss", cfg.seed, 12, H, T, "bf16", torch),
           "down_in": device_x("ffn_mid", cfg.seed, 13, F, T, "bf16", torch)}
    sets = []
    for r in range(ring):
        packed, alphas = {}, []
        for i, (n, (N, K)) in enumerate(shapes.items()):
            p, a = device_weights(N, K, 5000 + 10 * r + i, torch, hbl)
            packed[n] = p
            alphas.append(a)
        sets.append((packed, torch.cat(alphas)))
    dims = {"q": H, "k": H, "v": H, "o": H, "up": F, "gate": F, "down": H}
    outs = {n: torch.empty((T, d), dtype=torch.bfloat16, device="cuda") for n, d in dims.items()}
    work = hbl.new_workspace(hbl.hbl_block_workspace_bytes(T, H, F))
    state = {"i": 0, "path": hbl.PATH_AUTO}

    def call():
        r = state["i"] % ring
        state["i"] += 1
        hbl.hbl_block_forward(ins, sets[r][0], sets[r][1], H, F, 4, EPS, outputs=outs, workspace=work, path=state["path"])

    ms_b2b = None
    if small:
        ms = graph_ms(call, ring, iters or 10, torch)
        state["i"], state["path"] = 0, hbl.PATH_STREAM      # ordinary launches, for comparison (see layer_point)
        ms_b2b = graph_ms(call, ring, iters or 10, torch)
    else:
        flops = 2.0 * T * sum(n * k for n, k in shapes.values())
        est_ms = flops / 2.0e15 * 1e3
        ms = time_loop(call, iters or int(max(3, min(30, 300.0 / est_ms))), 2, torch)
    st = hbl.hbl_check_status()
    if st != 0:
        raise RuntimeError(f"device status {st} in block T={T}")
    ops = 2.0 * T * sum(n * k for n, k in shapes.values())
    tops = ops / (ms * 1e-3) / 1e12
    gbs = per_call / (ms * 1e-3) / 1e9
    out = {"point": "config5_block_7B", "tokens": T, "ms": round(ms, 5), "tokens_per_s": round(T / (ms * 1e-3), 1),
           "tops": round(tops, 2), "alg_gbs": round(gbs, 1), "ring": ring, "graph": small}
    if tops < 100 or small:
        out["bound"] = "hbm"; out["frac"] = round(gbs / peaks["hbm_gbs"], 4)
        out["frac_of_nominal_hbm"] = round(gbs / NOMINAL_HBM_GBS, 4)
        if ms_b2b is not None:
            out["ms_ordinary_launches"] = round(ms_b2b, 5)
            out["frac_ordinary_launches"] = round(per_call / (ms_b2b * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)
    else:
        out["bound"] = "tensor"; out["frac"] = round(tops / (2 * peaks["bf16_tflops"]), 4)
        out["frac_of_sustained"] = round(tops / (2 * peaks["bf16_tflops_sustained"]), 4)
        out["frac_of_nominal_int8"] = round(tops / NOMINAL_INT8_TOPS, 4)
    del ins, sets, outs, work
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------- CPU oracle legs
HEAD = dict(name="config3_Wdown_1p3B", kind="ffn_mid", seed=3, K=8192, N=2048, bits=4, had=True, T=16384)


def headline_config(world: int) -> dict:
    """The `config` object of the JSON line: the same in both arms (the reference arm times a bounded sample of it)."""
    h = HEAD
    return {"workload": f"{h['name']}: H-BitLinear in 8192 -> out 2048, INT4 activations + Hadamard, "
                        f"{h['T']} tokens per step, bf16 activations SiLU(a)*b with 0.2% outlier channels x40, "
                        f"ternary weights from N(0,0.02) latents",
            "l2": "two alternating 268 MB input batches (each larger than the 126 MB L2)",
            "parallelism": "replicas" if world > 1 else "single GPU"}


def oracle_rate(target_s=12.0):
    """Times the oracle as it stands on a bounded token sample of the headline workload."""
    from oracle import hbl_oracle as orc
    from paper_2504_18415_b200 import workloads as wl
    cores = orc.num_threads()
    cfg = wl.CONFIG3
    wt, alpha = orc.weight_quant(cfg.w_latent(), EPS, 32)
    n0 = max(cores, 8)
    x = cfg.x(0, n0)
    t0 = time.perf_counter()
    orc.forward(x, wt, alpha, cfg.bits, True, EPS, 32)
    dt = time.perf_counter() - t0
    n = int(max(n0, min(4096, n0 * target_s / max(dt, 1e-3))))
    n = (n // cores) * cores or cores
    x = cfg.x(0, n)
    t0 = time.perf_counter()
    orc.forward(x, wt, alpha, cfg.bits, True, EPS, 32)
    dt = time.perf_counter() - t0
    return {"value": round(n / dt, 2), "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"{n} tokens of {HEAD['name']} (in 8192 -> out 2048, INT4+Hadamard), all outputs, {dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import hbl_oracle as orc
    from paper_2504_18415_b200 import workloads as wl
    cores = orc.num_threads()
    cfg = wl.CONFIG3
    wt, alpha = orc.weight_quant(cfg.w_latent(), EPS, 32)
    n = max(cores, 16) * 4
    x = cfg.x(0, n)
    for _ in range(max(1, min(args.warmup, 3))):
        orc.forward(x[:cores], wt, alpha, cfg.bits, True, EPS, 32)
    t0 = time.perf_counter()
    steps = max(1, min(args.steps, 20))
    for _ in range(steps):
        orc.forward(x, wt, alpha, cfg.bits, True, EPS, 32)
    dt = (time.perf_counter() - t0) / steps
    val = n / dt
    sample = f"each step = {n} tokens of {HEAD['name']} through the CPU oracle (all 2048 outputs)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(val, 2), "unit": UNIT,
        "n_gpus": args.gpus, "steps": steps, "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": headline_config(int(os.environ.get("WORLD_SIZE", "1"))),
        "cpu_baseline": {"value": round(val, 2), "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(val, 2), "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- main (GPU arm)
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", default="quick", choices=["none", "quick", "full"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only", default="", help="comma-separated point filters 'name-substring:tokens' "
                    "(e.g. config4_a8_N32768:16,block:1); the sweep then runs just those points")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    from paper_2504_18415_b200 import hbl, workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks, peak_src = load_peaks()
    W = max(args.warmup, 3)
    Ksteps = max(args.steps, 1)

    # ---- headline workload: config 3 at T = 16384, full host-generated seeded inputs ----
    h = HEAD
    T, K, N = h["T"], h["K"], h["N"]
    cfg = wl.CONFIG3
    x_host = torch.from_numpy(cfg.x(0, T)).to(torch.bfloat16)
    xs = [x_host.cuda(), torch.roll(x_host, 1, 0).cuda()]            # two 268 MB inputs: every step is L2-cold
    packed, alpha = hbl.hbl_quantize_weights(torch.from_numpy(cfg.w_latent()).cuda(), EPS)
    ys = [torch.empty((T, N), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    work = hbl.new_workspace(hbl.hbl_workspace_bytes(T, K, N))

    def step(i):
        hbl.hbl_forward(xs[i & 1], packed, alpha, N, h["bits"], h["had"], EPS, y=ys[i & 1], workspace=work)

    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = hbl.hbl_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    # both kernels of the step are bracketed by events inside the timed region itself, so the per-kernel times
    # below belong to the same clocks as ms_per_step
    with hbl.KernelTimer(Ksteps, 2) as kt, hbl.KernelTimer(Ksteps, 1) as kt_act:
        e0.record()
        for i in range(Ksteps):
            step(i)
        e1.record()
        torch.cuda.synchronize()
    launches = hbl.hbl_launch_count() - launches0
    total_ms = e0.elapsed_time(e1)
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    torch.cuda.synchronize()
    # keep the GPU busy a little longer so that the clock sampler sees load
    if rank == 0:
        t_end = time.time() + 0.6
        i = 0
        while time.time() < t_end:
            step(i); i += 1
        torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    gemm_ms = statistics.mean(kt.times_ms())
    act_ms_timed = statistics.mean(kt_act.times_ms())
    st = hbl.hbl_check_status()
    if st != 0:
        raise RuntimeError(f"device status {st}")
    ms_per_step = total_ms / Ksteps
    value = whole_job_value(world, T, ms_per_step)

    # per-kernel breakdown: the two kernels on the caller's stream from the timed region; their sum is below
    # ms_per_step only by the gaps between launches (the weight expansion runs underneath the quantizer)
    breakdown = {"act_quant_kernel": round(act_ms_timed, 5), "gemm_tensor_kernel": round(gemm_ms, 5)}
    # Inside a step the weight expansion runs on the library's side stream underneath the quantizer, so its
    # own duration is taken from stand-alone launches of the same kernel.
    with hbl.KernelTimer(5, 3) as k2:
        for i in range(5):
            hbl.hbl_unpack_weights(packed, N, K)
    breakdown["unpack_kernel"] = round(statistics.mean(k2.times_ms()), 5)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- e2e: same call, host-resident x and y, copies inside the timed region ----
    xh = x_host.pin_memory()
    yh = torch.empty((T, N), dtype=torch.bfloat16).pin_memory()
    for i in range(2):
        hbl.hbl_forward_host(xh, packed, alpha, N, h["bits"], h["had"], yh, xs[0], ys[0], work)
    torch.cuda.synchronize()
    n_e2e = min(Ksteps, 10)
    t0 = time.perf_counter()
    for i in range(n_e2e):
        hbl.hbl_forward_host(xh, packed, alpha, N, h["bits"], h["had"], yh, xs[0], ys[0], work)
        torch.cuda.synchronize()
        _ = float(yh[0, 0])                                           # the host reads the step's result
    e2e_ms = (time.perf_counter() - t0) * 1e3 / n_e2e
    e2e = {"value": round(T / (e2e_ms * 1e-3), 1), "unit": "tokens/s", "h2d_bytes_per_step": T * K * 2,
           "d2h_bytes_per_step": T * N * 2, "ms_per_step": round(e2e_ms, 3), "steps": n_e2e}

    # the same step with the INT4 codes kept two per byte between the two kernels (half the code traffic; the
    # contraction widens them on the fly): reported beside the headline, which uses the faster one-per-byte form
    pk_state = {"i": 0}

    def step_packed():
        i = pk_state["i"]
        pk_state["i"] += 1
        hbl.hbl_forward(xs[i & 1], packed, alpha, N, h["bits"], h["had"], EPS, y=ys[i & 1], workspace=work,
                        path=hbl.PATH_TENSOR_PACKED)

    variants = {"int4_codes_two_per_byte_ms_per_step": round(time_loop(step_packed, min(Ksteps, 10), 3, torch), 5)}

    ops = 2.0 * T * K * N
    ach = ops / (gemm_ms * 1e-3) / 1e12
    step_tops = ops / (ms_per_step * 1e-3) / 1e12
    peak_i8 = 2.0 * peaks["bf16_tflops"]
    roofline = {"kernel": "gemm_tensor_kernel (tcgen05.mma kind::i8, 128x256x128 tiles)", "bound": "tensor",
                "achieved": round(ach, 2), "peak": round(peak_i8, 1), "unit": "TFLOP/s", "frac": round(ach / peak_i8, 4),
                "traffic": GEMM_TENSOR_TRAFFIC_BYTES,
                "traffic_source": "constant from one ncu capture of this kernel at this workload, not re-measured by this run",
                "frac_of_nominal_int8": round(ach / NOMINAL_INT8_TOPS, 4),
                "frac_of_library_int8": None,                      # filled in after the sweep (see below)
                # the whole step (quantizer + contraction), which is what the >= 0.60 target at >= 8192 tokens is about
                "step": {"tops": round(step_tops, 2), "frac_of_2x_bf16_measured": round(step_tops / peak_i8, 4),
                         "frac_of_nominal_int8": round(step_tops / NOMINAL_INT8_TOPS, 4),
                         "frac_of_library_int8": None,
                         "target_0p60_of_nominal_int8_met": bool(step_tops / NOMINAL_INT8_TOPS >= 0.60)},
                "note": f"int8 multiply-add = 2 ops; peak = 2 x {peak_src} bf16 burst (nominal int8:bf16 ratio), of measured; "
                        f"kernel avg {gemm_ms * 1e3:.1f} us over {len(kt.times_ms())} launches inside the timed region"}
    act_ms = breakdown["act_quant_kernel"]
    kernels = {
        "fwht_quant_bf16_kernel": {
            "ms": act_ms, "hbm_gbs": round(3.0 * T * K / (act_ms * 1e-3) / 1e9, 1),
            "hbm_frac": round(3.0 * T * K / (act_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
            "alu_frac": round(12.5 * T * K / (act_ms * 1e-3) / ALU_PEAK_LANE_OPS, 4),
            "note": "3 B of kernel traffic and 12.5 fp32 lane-ops per element; ALU peak 148 SMs x 128 lanes x 1.965 GHz"},
        "unpack_kernel": {"ms": breakdown["unpack_kernel"],
                          "hbm_frac": round(1.25 * N * K / (breakdown["unpack_kernel"] * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                          "note": "timed alone; inside the step it overlaps the quantizer on a side stream"},
        "gemm_tensor_kernel": {"ms": breakdown["gemm_tensor_kernel"]},
    }

    points = []
    if args.sweep != "none" and world == 1:
        del xs, ys, work
        torch.cuda.empty_cache()
        full = args.sweep == "full"
        only = [f.split(":") for f in args.only.split(",") if f]
        want = lambda name, T_: (not only) or any(o[0] in name and (len(o) < 2 or int(o[1]) == T_) for o in only)

        # layer and block points are listed in the order they are printed in, but the ones of up to 512 tokens
        # (latency- and HBM-bound) are measured before the long tensor-bound ones, which leave the clocks under the
        # power cap for a while
        plan = []

        def L(name, kind, seed, K_, N_, bits, had, T_):
            if want(name, T_):
                plan.append((T_, lambda: layer_point(name, kind, seed, K_, N_, bits, had, T_, torch=torch, hbl=hbl, peaks=peaks)))

        # the activation-side kernels first: they are bound by instruction issue, and right after the
        # millisecond-long contractions below the power cap still holds the clocks down
        if full:
            for dtype_name in ("f32", "bf16"):
                for N_, K_ in ((2048, 8192), (4096, 16384)):            # W_down of the 1.3B and the 7B configuration
                    if want(f"weight_quantize_{dtype_name}", 0):
                        points.append(weight_quantize_point(N_, K_, dtype_name, torch, hbl, peaks))
            for bits_ in (8, 4):
                if want(f"row_quantize_int{bits_}", 32768):
                    points.append(row_quantize_point(4096, 32768, bits_, torch, hbl, peaks))
            for bits_ in (3, 4):
                if want(f"kv_quantize_int{bits_}", 16384):
                    points.append(kv_quantize_point(16384, 32, 128, bits_, torch, hbl, peaks))    # one of K / V of the 7B shape
            for K_ in (4096, 8192):
                if want("transform_backward_bf16", 16384):
                    points.append(backward_transform_point(K_, 16384, torch, hbl, peaks))
                if want("norm_transform_quantize_int4", 16384):
                    points.append(norm_quantize_point(K_, 16384, torch, hbl, peaks))
                if want("glu_transform_quantize_int4", 16384):
                    points.append(glu_quantize_point(K_, 16384, torch, hbl, peaks))
        for T_ in (1, 16, 256, 4096):
            L("config2_Wo_1p3B", "attn_out", 2, 2048, 2048, 4, True, T_)
        for T_ in (1, 16, 1024):
            L("config3_Wdown_1p3B", "ffn_mid", 3, 8192, 2048, 4, True, T_)
        for N_ in (12288, 32768):
            for T_ in (16, 4096, 32768):
                L(f"config4_a8_N{N_}", "gauss", 4, 4096, N_, 8, False, T_)
        for T_ in ((1, 4, 16, 64, 256, 1024, 4096, 16384, 65536) if full else (1, 16, 256, 4096, 16384)):
            if want("config5_block_7B", T_):
                plan.append((T_, lambda T_=T_: block_point(T_, torch, hbl, peaks)))
        results = [None] * len(plan)
        for small_first in (True, False):
            for i, (T_, run) in enumerate(plan):
                if (T_ <= 512) == small_first:
                    results[i] = run()
        points.extend(results)

    # the library int8 GEMM runs last: seconds of back-to-back tensor work leave the clocks under the power cap,
    # which the issue-bound points of the sweep would otherwise inherit
    lib_i8 = library_int8_peak(torch)
    if lib_i8["int8_library_tops_burst"]:
        roofline["frac_of_library_int8"] = round(ach / lib_i8["int8_library_tops_burst"], 4)
        roofline["step"]["frac_of_library_int8"] = round(step_tops / lib_i8["int8_library_tops_burst"], 4)

    cpu = None
    if not args.no_cpu_baseline:
        cpu = oracle_rate()

    out = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": Ksteps, "warmup": W,
        "ms_per_step": round(ms_per_step, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "s8", "data": "synthetic",
        "config": headline_config(world),
        "tops": round(ops / (ms_per_step * 1e-3) / 1e12, 2),
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "kernels_ms": breakdown, "kernels": kernels, "variants": variants, "roofline": roofline, "cpu_baseline": cpu, "points": points,
        "peaks": {**peaks, "source": peak_src, "int8_nominal_tops": NOMINAL_INT8_TOPS, "hbm_nominal_gbs": NOMINAL_HBM_GBS,
                  **lib_i8},
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
