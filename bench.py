#!/usr/bin/env python
"""Benchmark of the HiF8 conversion hot path on B200.

One step = per-tensor scaled encode (amax -> power-of-two scale -> HiF8 bytes, just-in-time form) followed
by decode back to FP32 of one FP32 4096x4096 N(0,1) tensor (synthetic, seeded).  The metric is algorithmic
bytes moved per second: 9 B/element for the encode call (4 read for amax, 4 read + 1 written for the
conversion) plus 5 B/element for the decode call (1 read, 4 written).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 is launched under torch.distributed.run, one rank per GPU; ranks convert independent tensors (no
data-path collective, weak scaling) and rank 0 prints the single JSON line.
`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

ROWS, COLS = 4096, 4096
N_EL = ROWS * COLS
BYTES_ENCODE = 9 * N_EL   # amax read + conversion read + byte write
BYTES_DECODE = 5 * N_EL
BYTES_STEP = BYTES_ENCODE + BYTES_DECODE
POOL = 6                  # rotating buffer sets: 6 x 64 MiB of input alone exceeds the 126 MB L2
WORKLOAD = "fp32_4096x4096_normal_amax_scale_encode_then_decode"
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu capture summarised in profiles/;
# None for a kernel changed since its capture
TRAFFIC = {"amax_kernel<f32>": 67.57e6, "convert_kernel<f32,TA>": 69.53e6, "decode_kernel<f32>": 26.10e6}
METRIC = "hif8_encode_decode_throughput"
UNIT = "GB/s"


def env_int(name, default):
    try:
        return int(os.environ.get(name, default))
    except ValueError:
        return default


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without an initialised process group)."""
    if dist is None or not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def job_throughput(world, bytes_per_rank_step, ms_per_step):
    """Whole-job GB/s: every rank converts its own tensor (weak scaling), time is the slowest rank's."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def cpu_baseline(sample_elems):
    """The oracle as it stands (brute-force nearest-of-256 encode), on a leading slice of the same tensor."""
    from oracle import hif8_oracle as O
    x = W.normal_f32((ROWS, COLS), seed=1234).reshape(-1)[:sample_elems]
    t0 = time.perf_counter()
    _, se = O.amax_scale(x, O.F32, 14)
    codes = O.encode(x, O.F32, se, O.TA, 0, quick=False)
    O.decode(codes, O.F32, se)
    dt = time.perf_counter() - t0
    return {"value": 14 * sample_elems / dt / 1e9, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
            "sample": f"first {sample_elems} of {N_EL} elements: amax + brute-force TA encode + decode, {dt:.2f} s",
            "elements_per_s": sample_elems / dt}


def extra_results(H, torch, hbm_peak, peak_kind):
    """Secondary workloads (each with its own roofline fraction): BF16 fake-quant of an LLM-activation tensor,
    gradient-range FP32 encode/decode, and the HiF8-operand GEMM.  Inputs are generated on the device from a
    seeded torch generator with the same recipes as workloads/ (shapes and distributions, not the same bytes)."""
    out = {}
    g = torch.Generator(device="cuda")
    g.manual_seed(2345)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wsb = H.hif8_workspace_bytes(H.WS_FAKE_QUANT, 0)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")

    def timed(fn, reps):
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        ev0.record()
        for r in range(reps):
            fn(r)
        ev1.record()
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1) / reps

    # ---- small and odd sizes (launch latency, tails): FP32 encode TA + decode, 20 call pairs per graph replay
    small = {}
    for n in (9408, 1000003, 4096 * 11008, 256 * 64 * 56 * 56):
        xs_ = torch.randn(n, generator=g, device="cuda")
        cq = torch.empty(n, dtype=torch.uint8, device="cuda")
        bk = torch.empty(n, dtype=torch.float32, device="cuda")
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            cs = torch.cuda.current_stream().cuda_stream
            for _ in range(20):
                H.hif8_encode(xs_, H.F32, cq, n, 10, H.RND_TA, stream=cs)
                H.hif8_decode(cq, bk, H.F32, n, 10, stream=cs)
        ms = timed(lambda r: gr.replay(), 5) / 20
        small[str(n)] = {"us_per_encode_decode_pair": ms * 1e3, "GBps": 10 * n / ms / 1e6, "frac": 10 * n / ms / 1e6 / hbm_peak}
        del xs_, cq, bk, gr
    out["small_and_odd_sizes_f32"] = {"bytes_per_element": 10, "sizes": small, "peak": hbm_peak, "peak_kind": f"of {peak_kind}",
                                      "note": "tensors up to 45 M elements fit in L2 between the two calls; a pair is two launches"}

    # ---- LLM-activation fake-quant: BF16 [8192 x 8192], Student-t(3) body, 0.1 % of channels x100
    T = Hd = 8192
    n = T * Hd
    xs = []
    for _ in range(2):
        z = torch.randn(T, Hd, generator=g, device="cuda")
        chi = torch.zeros_like(z)
        for _ in range(3):
            chi += torch.randn(T, Hd, generator=g, device="cuda") ** 2
        x = z / torch.sqrt(chi / 3.0)
        cols = torch.randperm(Hd, generator=g, device="cuda")[:8]
        x[:, cols] *= 100.0
        xs.append(x.to(torch.bfloat16))
        del z, chi, x
    ys = [torch.empty_like(x) for x in xs]
    fq = {}
    for name, mode in (("TA", H.RND_TA), ("HR", H.RND_HR), ("SSR", H.RND_SSR), ("TE", H.RND_TE), ("SR", H.RND_SR)):
        ms = timed(lambda r: H.hif8_fake_quant(xs[r & 1], ys[r & 1], H.BF16, n, 1, 14, mode, 0, 7, None, None, ws, wsb), 20)
        fq[name] = {"ms": ms, "GBps": 6 * n / ms / 1e6, "frac": 6 * n / ms / 1e6 / hbm_peak}
    ms = timed(lambda r: H.hif8_fake_quant(xs[r & 1], ys[r & 1], H.BF16, n, 0, 3, H.RND_TA, 0, 0), 20)
    fq["TA_given_scale"] = {"ms": ms, "GBps": 4 * n / ms / 1e6, "frac": 4 * n / ms / 1e6 / hbm_peak}
    # the same tensors to HiF8 bytes with a given scale (2 B read + 1 B written): forward (TA) and backward (HR) rounding
    cq = torch.empty(n, dtype=torch.uint8, device="cuda")
    enc = {}
    for name, mode in (("TA", H.RND_TA), ("HR", H.RND_HR)):
        ms = timed(lambda r: H.hif8_encode(xs[r & 1], H.BF16, cq, n, 3, mode), 20)
        enc[name] = {"ms": ms, "GBps": 3 * n / ms / 1e6, "frac": 3 * n / ms / 1e6 / hbm_peak}
    out["encode_bf16_8192x8192"] = {"bytes_per_element": 3, "modes": enc, "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
    del cq
    out["fake_quant_bf16_8192x8192"] = {"bytes_per_element": {"fused_amax": 6, "given_scale": 4}, "modes": fq,
                                        "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
    del xs, ys

    # ---- gradient-range stress: FP32 2^28 elements, log-uniform magnitudes 2^-40 .. 2^20, random signs
    n = 1 << 28
    e = torch.randint(-40, 20, (n,), generator=g, device="cuda", dtype=torch.int32) + 127
    m = torch.randint(0, 1 << 23, (n,), generator=g, device="cuda", dtype=torch.int32)
    sg = torch.randint(0, 2, (n,), generator=g, device="cuda", dtype=torch.int32)
    bits = (sg << 31) | (e << 23) | m
    del e, m, sg
    codes = torch.empty(n, dtype=torch.uint8, device="cuda")
    back = torch.empty(n, dtype=torch.float32, device="cuda")
    res = {}
    for name, mode in (("encode_TA", H.RND_TA), ("encode_HR", H.RND_HR)):
        ms = timed(lambda r: H.hif8_encode(bits, H.F32, codes, n, 0, mode), 10)
        res[name] = {"ms": ms, "GBps": 5 * n / ms / 1e6, "frac": 5 * n / ms / 1e6 / hbm_peak}
    ms = timed(lambda r: H.hif8_decode(codes, back, H.F32, n, 0), 10)
    res["decode"] = {"ms": ms, "GBps": 5 * n / ms / 1e6, "frac": 5 * n / ms / 1e6 / hbm_peak}
    out["loguniform_f32_2^28"] = {"bytes_per_element": 5, "calls": res, "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
    del bits, codes, back

    # ---- GEMM: A BF16 8192x8192 N(0,1), W BF16 8192x28672 N(0,0.02), per-tensor scaled to HiF8, C = dec(A) dec(W)
    M, N, K = 8192, 28672, 8192
    a = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
    w = (torch.randn(K, N, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    Aq = torch.empty(M * K, dtype=torch.uint8, device="cuda")
    Wq = torch.empty(K * N, dtype=torch.uint8, device="cuda")
    se = torch.zeros(2, dtype=torch.int32, device="cuda")
    H.hif8_amax_scale_encode(a, H.BF16, Aq, M * K, 14, H.RND_TA, 0, 0, None, None, se[0:1], None, ws, wsb)
    H.hif8_amax_scale_encode(w, H.BF16, Wq, K * N, 14, H.RND_TA, 0, 0, None, None, se[1:2], None, ws, wsb)
    # per-channel weight scaling of the same weight (one exponent per output column / per row of the [N,K] view) and
    # the delayed-scaling cadence on the activation; bytes per element: source reads + code byte
    ch_amax = torch.empty(N, dtype=torch.float32, device="cuda")
    ch_se = torch.empty(N, dtype=torch.int32, device="cuda")
    ch_amax2 = torch.empty(2 * N, dtype=torch.float32, device="cuda")
    ch_se2 = torch.empty(2 * N, dtype=torch.int32, device="cuda")
    chan = {}
    ms = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, K, N, 1, 14, H.RND_TA, 0, 0, None, ch_amax, ch_se), 10)
    chan["columns_[K,N]"] = {"ms": ms, "bytes_per_element": 5, "GBps": 5 * K * N / ms / 1e6, "frac": 5 * K * N / ms / 1e6 / hbm_peak,
                             "note": "amax kernel (2 B) + encode kernel (2 + 1 B)"}
    ms = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, N, K, 0, 14, H.RND_TA, 0, 0, None, ch_amax, ch_se), 10)
    chan["rows_[N,K]"] = {"ms": ms, "bytes_per_element": 3, "GBps": 3 * K * N / ms / 1e6, "frac": 3 * K * N / ms / 1e6 / hbm_peak,
                          "note": "one kernel, a block per row; the second read of the row hits L1/L2"}
    ms = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, 2 * N, K // 2, 0, 14, H.RND_TA, 0, 0, None, ch_amax2, ch_se2), 10)
    chan["rows_[2N,K/2]"] = {"ms": ms, "bytes_per_element": 3, "GBps": 3 * K * N / ms / 1e6, "frac": 3 * K * N / ms / 1e6 / hbm_peak,
                             "note": "rows of 4096: two rows per block"}
    ms = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, N // 2, 2 * K, 0, 14, H.RND_TA, 0, 0, None, ch_amax2, ch_se2), 10)
    chan["rows_[N/2,2K]"] = {"ms": ms, "bytes_per_element": 3, "GBps": 3 * K * N / ms / 1e6, "frac": 3 * K * N / ms / 1e6 / hbm_peak,
                             "note": "rows of 16384: held in registers, read once"}
    ms = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, K, N, 1, 14, H.RND_TA, 0, 0, ch_se, None, None), 10)
    chan["columns_given_exponents"] = {"ms": ms, "bytes_per_element": 3, "GBps": 3 * K * N / ms / 1e6,
                                       "frac": 3 * K * N / ms / 1e6 / hbm_peak}
    out["channel_scaled_encode_bf16_8192x28672"] = {"calls": chan, "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
    state = torch.empty(H.SCALE_STATE_BYTES, dtype=torch.uint8, device="cuda")
    H.hif8_scale_state_init(state, 4)
    dl = {}
    for name, measure in (("measuring_iteration", 1), ("plain_iteration", 0)):
        ms = timed(lambda r: H.hif8_delayed_scale_encode(a, H.BF16, Aq, M * K, H.RND_TA, 0, 0, state, measure, 14), 20)
        dl[name] = {"ms": ms, "GBps": 3 * M * K / ms / 1e6, "frac": 3 * M * K / ms / 1e6 / hbm_peak}
    ms = timed(lambda r: H.hif8_encode_transpose(a, H.BF16, Aq, M, K, 3, None, H.RND_HR), 20)
    out["encode_transpose_bf16_8192x8192_HR"] = {"ms": ms, "bytes_per_element": 3, "GBps": 3 * M * K / ms / 1e6,
                                                 "frac": 3 * M * K / ms / 1e6 / hbm_peak, "peak": hbm_peak,
                                                 "peak_kind": f"of {peak_kind}"}
    out["delayed_scale_encode_bf16_8192x8192"] = {"bytes_per_element": 3, "calls": dl, "peak": hbm_peak,
                                                  "peak_kind": f"of {peak_kind}"}
    H.hif8_amax_scale_encode(a, H.BF16, Aq, M * K, 14, H.RND_TA, 0, 0, None, None, se[0:1], None, ws, wsb)
    H.hif8_amax_scale_encode(w, H.BF16, Wq, K * N, 14, H.RND_TA, 0, 0, None, None, se[1:2], None, ws, wsb)
    del a, w
    C = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    gws_b = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N)
    gws = torch.empty(gws_b, dtype=torch.uint8, device="cuda")
    tf_peak, tf_kind = 1590.0, "fallback"
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        tf_peak, tf_kind = float(json.load(open(path))["bf16_tflops"]), "measured"
    flops = 2.0 * M * N * K
    ms = timed(lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, gws_b), 10)
    st1 = H.hif8_gemm_status(gws)
    ms_f = timed(lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, 256), 3)
    st2 = H.hif8_gemm_status(gws)
    ch_se.fill_(int(se[1]))
    ms_c = timed(lambda r: H.hif8_gemm_channel_scaled(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], ch_se, gws, gws_b), 10)
    st3 = H.hif8_gemm_status(gws)
    # backward-pass forms of the same size: dgrad reads the weight as [N,K], wgrad reads A as [K,M] and accumulates in FP32
    bw = {}
    ms_d = timed(lambda r: H.hif8_gemm_ex(Aq, K, 0, Wq, K, 1, C, N, H.BF16, M, N, K, se[0:1], se[1:2], None, 0, gws, gws_b), 10)
    bw["dgrad_form_w_as_[N,K]"] = {"ms": ms_d, "TFLOPs": flops / ms_d / 1e9, "frac": flops / ms_d / 1e9 / tf_peak,
                                   "device_status": H.hif8_gemm_status(gws)}
    C32 = torch.zeros(M, N, dtype=torch.float32, device="cuda")
    ms_w = timed(lambda r: H.hif8_gemm_ex(Aq, M, 1, Wq, N, 0, C32, N, H.F32, M, N, K, se[0:1], se[1:2], None, 1, gws, gws_b), 10)
    bw["wgrad_form_a_as_[K,M]_fp32_accumulate"] = {"ms": ms_w, "TFLOPs": flops / ms_w / 1e9, "frac": flops / ms_w / 1e9 / tf_peak,
                                                   "device_status": H.hif8_gemm_status(gws)}
    del C32
    # inference-decode shapes: a few activation rows against the same weight (bound by reading the weight bytes once)
    narrow = {}
    for Mn in (16, 64):
        Cn = torch.empty(Mn, N, dtype=torch.bfloat16, device="cuda")
        # with the workspace: equal (slab, k-block) ranges per SM; with the 256-byte minimum: one CTA per slab
        ms_n = timed(lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, Cn, N, H.BF16, Mn, N, K, se[0:1], se[1:2], gws, gws_b), 20)
        ms_s = timed(lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, Cn, N, H.BF16, Mn, N, K, se[0:1], se[1:2], gws, 256), 20)
        byt = K * N + Mn * K + 2 * Mn * N
        narrow[f"M={Mn}"] = {"us": ms_n * 1e3, "GBps": byt / ms_n / 1e6, "frac_of_hbm": byt / ms_n / 1e6 / hbm_peak,
                             "us_one_cta_per_slab": ms_s * 1e3, "device_status": H.hif8_gemm_status(gws)}
        del Cn
    out["gemm_narrow_Mx28672x8192"] = {"bound": "hbm", "bytes": "K*N weight bytes + M*K + 2*M*N", "shapes": narrow,
                                       "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
    out["gemm_8192x28672x8192"] = {
        "backward_forms": bw,
        "decode_once_channel_scaled": {"ms": ms_c, "TFLOPs": flops / ms_c / 1e9, "frac": flops / ms_c / 1e9 / tf_peak,
                                       "device_status": st3, "note": "one weight exponent per output column"},
        "decode_once": {"ms": ms, "TFLOPs": flops / ms / 1e9, "frac": flops / ms / 1e9 / tf_peak, "device_status": st1,
                        "note": "whole call: decode of both operands to BF16 workspace + tcgen05 kernel"},
        "fused": {"ms": ms_f, "TFLOPs": flops / ms_f / 1e9, "frac": flops / ms_f / 1e9 / tf_peak, "device_status": st2,
                  "note": "no workspace: byte tiles decoded per CTA in shared memory"},
        "bound": "tensor", "peak": tf_peak, "peak_kind": f"of {tf_kind} (cuBLAS BF16 burst)", "unit": "TFLOP/s",
        "scale_exps": [int(v) for v in se.cpu()], "output": "bf16"}
    del C, gws, Aq, Wq

    # ---- Algorithm 1, one layer: 10 x 10 grid of scale exponents, 4096^3 (20 casts, 100 GEMMs, 100 MSE reductions)
    M = N = K = 4096
    a = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
    w = (torch.randn(K, N, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    o_ref = torch.matmul(a.float(), w.float())
    pb = H.hif8_pts_workspace_bytes(M, N, K, 10)
    pws = torch.empty(pb, dtype=torch.uint8, device="cuda")
    d_err = torch.zeros(100, dtype=torch.float32, device="cuda")
    d_best = torch.zeros(2, dtype=torch.int32, device="cuda")
    ms = timed(lambda r: H.hif8_pts_search(a, w, H.BF16, 0, o_ref, N, M, N, K, -4, 5, d_err, d_best, pws, pb), 3)
    out["pts_search_4096^3"] = {"ms": ms, "TFLOPs_of_100_gemms": 100 * 2.0 * M * N * K / ms / 1e9,
                                "best_exponents": [int(v) for v in d_best.cpu()], "device_status": H.hif8_pts_status(pws),
                                "min_mse": float(d_err.min().item())}
    return out


def run_reference(args, rank):
    if rank != 0:
        return
    from oracle import hif8_oracle as O
    sample = 1 << 20
    x = W.normal_f32((ROWS, COLS), seed=1234).reshape(-1)[:sample]

    def step():
        _, se = O.amax_scale(x, O.F32, 14)
        codes = O.encode(x, O.F32, se, O.TA, 0, quick=False)
        O.decode(codes, O.F32, se)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    value = 14 * sample / dt / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": f"first {sample} of {N_EL} elements per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
                             "sample": f"first {sample} of {N_EL} elements per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the secondary workloads (fake-quant, 2^28 stress, GEMM)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    rank, world, local = env_int("RANK", 0), env_int("WORLD_SIZE", 1), env_int("LOCAL_RANK", 0)

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    import paper_2409_16626_b200 as H

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # ---- synthetic inputs: POOL independent N(0,1) tensors per rank, resident in HBM
    srcs = [torch.from_numpy(W.normal_f32((ROWS, COLS), seed=1234 + 100 * rank + i)).cuda() for i in range(POOL)]
    codes = [torch.empty(N_EL, dtype=torch.uint8, device="cuda") for _ in range(POOL)]
    backs = [torch.empty(N_EL, dtype=torch.float32, device="cuda") for _ in range(POOL)]
    wsb = H.hif8_workspace_bytes(H.WS_AMAX_SCALE_ENCODE, N_EL)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")
    scal = torch.zeros(4, dtype=torch.int32, device="cuda")   # amax, scale_exp, scale
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream

    def encode_call(i):
        H.hif8_amax_scale_encode(srcs[i], H.F32, codes[i], N_EL, 14, H.RND_TA, 0, 0, None, scal[0:1], scal[1:2], scal[2:3],
                                 ws, wsb, stream=sp)

    def decode_call(i, se):
        H.hif8_decode(codes[i], backs[i], H.F32, N_EL, se, stream=sp)

    encode_call(0)
    torch.cuda.synchronize()
    se = int(scal[1].item())   # same distribution for every tensor of the pool: the descale exponent is fixed up front

    for w in range(args.warmup):
        encode_call(w % POOL)
        decode_call(w % POOL, se)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: device-resident inputs, CUDA events on the launching stream.
    # The launch sequence of POOL consecutive steps (one per buffer set) is captured once in a CUDA graph and
    # replayed, so the host's per-launch cost stays out of the device timeline; K steps = K // POOL replays of that
    # graph plus one replay of a second graph holding the remaining K % POOL steps, so exactly K steps are timed.
    K = max(1, args.steps)
    W_REPLAYS = max(1, -(-args.warmup // POOL))   # warm-up in whole replays: at least args.warmup steps
    ws2 = [ws, torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")]
    scal2 = [scal, torch.zeros(4, dtype=torch.int32, device="cuda")]

    def capture(two_streams, nsteps=POOL):
        """nsteps consecutive steps in one graph.  With two_streams, even and odd steps (independent tensors, separate
        workspaces) are enqueued on two streams, so the ramp and drain of one step's kernels overlap the other's."""
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            main_s = torch.cuda.current_stream()
            side_s = torch.cuda.Stream() if two_streams else main_s
            if two_streams:
                side_s.wait_stream(main_s)
            for i in range(nsteps):
                st = (main_s, side_s)[i & 1]
                cs = st.cuda_stream
                H.hif8_amax_scale_encode(srcs[i], H.F32, codes[i], N_EL, 14, H.RND_TA, 0, 0, None, scal2[i & 1][0:1],
                                         scal2[i & 1][1:2], scal2[i & 1][2:3], ws2[i & 1], wsb, stream=cs)
                H.hif8_decode(codes[i], backs[i], H.F32, N_EL, se, stream=cs)
            if two_streams:
                main_s.wait_stream(side_s)
        return gr

    def replay_steps(gr, tail):
        for _ in range(K // POOL):
            gr.replay()
        if tail is not None:
            tail.replay()

    def time_graph(gr, tail):
        for _ in range(W_REPLAYS):
            gr.replay()
        if tail is not None:
            tail.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        replay_steps(gr, tail)
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / K

    # one stream: every kernel waits for the previous one to drain
    serial_ms = time_graph(capture(False), capture(False, K % POOL) if K % POOL else None)
    graph = capture(True)
    graph_tail = capture(True, K % POOL) if K % POOL else None
    for _ in range(W_REPLAYS):
        graph.replay()
    if graph_tail is not None:
        graph_tail.replay()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with ClockSampler(local) as clk:
        t0.record(stream)
        replay_steps(graph, graph_tail)
        t1.record(stream)
        torch.cuda.synchronize()
        # per-kernel durations, measured live: each kernel of the step in a graph of its own (POOL launches over the
        # rotating buffers: hif8_amax -> the two-word clearing kernel + amax_kernel; hif8_encode with the scale known ->
        # the same convert_kernel the scaled call launches; hif8_decode -> decode_kernel), replayed between two events.
        # Direct launches would time the host's launch rate, not these ~15 us kernels.
        amax_out = torch.zeros(1, dtype=torch.float32, device="cuda")

        def kernel_ms(call):
            gk = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gk):
                cs = torch.cuda.current_stream().cuda_stream
                for i in range(POOL):
                    call(i, cs)
            R = max(4, min(K, 600) // POOL)   # own repeat count: these are per-kernel figures, not the timed K steps
            for _ in range(3):
                gk.replay()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(R):
                gk.replay()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / (R * POOL)

        amax_ms = kernel_ms(lambda i, cs: H.hif8_amax(srcs[i], H.F32, N_EL, amax_out, ws, wsb, stream=cs))
        conv_ms = kernel_ms(lambda i, cs: H.hif8_encode(srcs[i], H.F32, codes[i], N_EL, se, H.RND_TA, 0, 0, stream=cs))
        dec_ms = kernel_ms(lambda i, cs: H.hif8_decode(codes[i], backs[i], H.F32, N_EL, se, stream=cs))
        enc_ms = kernel_ms(lambda i, cs: H.hif8_amax_scale_encode(srcs[i], H.F32, codes[i], N_EL, 14, H.RND_TA, 0, 0, None,
                                                                  scal[0:1], scal[1:2], scal[2:3], ws, wsb, stream=cs))
    barrier()
    launches = 4 * K   # accumulator clear + amax + convert + decode kernels per step (graph replays)
    total_ms = t0.elapsed_time(t1)

    # ---- end to end: pinned host input -> device, both calls, results back to pinned host memory.  Consecutive
    # steps alternate between two streams (own host buffers, workspace and scalars each), so the upload of one step
    # overlaps the download of the previous one (PCIe is full duplex); every step still moves all its bytes.
    E = max(4, min(args.e2e_steps, K)) // 2 * 2
    lanes = []
    for j in range(2):
        lanes.append({
            "stream": torch.cuda.Stream(),
            "h_src": torch.from_numpy(W.normal_f32((ROWS, COLS), seed=999 + rank + j)).pin_memory(),
            "h_codes": torch.empty(N_EL, dtype=torch.uint8).pin_memory(),
            "h_back": torch.empty(N_EL, dtype=torch.float32).pin_memory(),
        })

    def e2e_step(k):
        ln, i = lanes[k & 1], k % POOL
        st = ln["stream"]
        with torch.cuda.stream(st):
            srcs[i].copy_(ln["h_src"], non_blocking=True)
            H.hif8_amax_scale_encode(srcs[i], H.F32, codes[i], N_EL, 14, H.RND_TA, 0, 0, None, scal2[k & 1][0:1],
                                     scal2[k & 1][1:2], scal2[k & 1][2:3], ws2[k & 1], wsb, stream=st.cuda_stream)
            H.hif8_decode(codes[i], backs[i], H.F32, N_EL, se, stream=st.cuda_stream)
            ln["h_codes"].copy_(codes[i], non_blocking=True)
            ln["h_back"].copy_(backs[i].view(-1), non_blocking=True)

    def e2e_run(n):
        for ln in lanes:
            ln["stream"].wait_stream(stream)
        for k in range(n):
            e2e_step(k)
        for ln in lanes:
            stream.wait_stream(ln["stream"])

    e2e_run(4)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    e2e_run(E)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / E

    total_ms, e2e_ms, enc_ms, dec_ms, amax_ms, conv_ms = max_over_ranks(
        [total_ms, e2e_ms, enc_ms, dec_ms, amax_ms, conv_ms], dist if world > 1 else None, "cuda")

    if rank == 0:
        ms_per_step = total_ms / K
        value = job_throughput(world, BYTES_STEP, ms_per_step)
        peak, peak_kind = load_peaks()
        kernels = {
            "amax_kernel<f32>": {"ms": amax_ms, "bytes": 4 * N_EL, "note": "hif8_amax call: accumulator-clearing kernel + amax kernel"},
            "convert_kernel<f32,TA>": {"ms": conv_ms, "bytes": 5 * N_EL},
            "decode_kernel<f32>": {"ms": dec_ms, "bytes": 5 * N_EL},
        }
        for kv in kernels.values():
            kv["GBps"] = kv["bytes"] / (kv["ms"] * 1e-3) / 1e9
            kv["frac"] = kv["GBps"] / peak
        # the dominant kernel: longest live duration among the single-kernel calls
        dom = max(("convert_kernel<f32,TA>", "decode_kernel<f32>"), key=lambda kname: kernels[kname]["ms"])
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "elements": N_EL, "rounding": "TA", "target_exp": 14,
                       "launch": f"CUDA graph of {POOL} steps replayed (+ one graph of steps % {POOL}); even/odd steps "
                                 "(independent tensors) on two streams",
                       "ms_per_step_single_stream": serial_ms,
                       "l2": f"inputs rotate over {POOL} buffer sets ({POOL * N_EL * 4 >> 20} MiB of sources) > 126 MB L2",
                       "bytes_per_step": BYTES_STEP, "elements_per_s": world * N_EL / (ms_per_step * 1e-3)},
            "clocks": clk.summary(),
            "e2e": {"value": job_throughput(world, BYTES_STEP, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": 4 * N_EL, "d2h_bytes_per_step": 5 * N_EL},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["GBps"], "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": kernels[dom]["frac"],
                         "traffic": TRAFFIC.get(dom), "algorithmic_bytes_per_launch": kernels[dom]["bytes"],
                         "avg_launch_ms": kernels[dom]["ms"]},
            "kernels": kernels,
            "calls": {"amax_scale_encode_ms": enc_ms, "amax_scale_encode_GBps": BYTES_ENCODE / (enc_ms * 1e-3) / 1e9},
        }
        if world == 1 and not args.no_extra:
            del srcs, codes, backs
            torch.cuda.empty_cache()
            line["extra"] = extra_results(H, torch, peak, peak_kind)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(1 << 23)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
