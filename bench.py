#!/usr/bin/env python
"""Benchmark of the HiF8 conversion hot path on B200.

One step = per-tensor scaled encode (amax -> power-of-two scale -> HiF8 bytes, just-in-time form) followed
by decode back to FP32 of one FP32 4096x4096 N(0,1) tensor (synthetic, seeded).  The metric is algorithmic
bytes moved per second: 9 B/element for the encode call (4 read for amax, 4 read + 1 written for the
conversion) plus 5 B/element for the decode call (1 read, 4 written).  It is NOT a DRAM bandwidth: the second
read of the source and the read of the codes can be served by the L2; `config.step_dram` gives the DRAM-based
figure from profiler counters beside it, and `roofline` describes single kernels.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
  python bench.py --case NAME [--reps R]        one named workload a few times, for use under a profiler

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
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from profiler captures of these kernels on this
# workload.  "cold": every launch alone with the caches flushed in front of it.  "in_step": the same launches inside the
# running amax -> convert -> decode sequence with the caches left as the previous kernel left them.  None: the kernel
# has changed since its capture.
TRAFFIC_COLD = {"amax_kernel<f32>": 67.14e6, "convert_kernel<f32,TA>": 67.38e6, "decode_kernel<f32>": 22.59e6}
TRAFFIC_IN_STEP = {"amax_kernel<f32>": 88.7e6, "convert_kernel<f32,TA>": 18.4e6, "decode_kernel<f32>": 52.5e6}
METRIC = "hif8_encode_decode_throughput"
UNIT = "GB/s"
MIN_REPEATS = 7


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


def spread(samples_ms):
    """median / best / worst of a list of per-unit times (ms)."""
    s = sorted(float(v) for v in samples_ms)
    return {"ms": s[len(s) // 2] if len(s) % 2 else 0.5 * (s[len(s) // 2 - 1] + s[len(s) // 2]), "best_ms": s[0],
            "worst_ms": s[-1], "repeats": len(s)}


def repeats_for(region_ms):
    """How often a timed region is repeated: at least MIN_REPEATS, more for short regions (about half a second of
    device time in all, so that the clock sampler sees the run), never more than 200."""
    return int(min(200, max(MIN_REPEATS, 500.0 / max(region_ms, 1e-3))))


def load_peaks():
    """(HBM GB/s, BF16 burst TFLOP/s, BF16 sustained TFLOP/s, kind)"""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), float(p["bf16_tflops"]), float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "measured"
    return 6650.0, 1590.0, 1400.0, "fallback"


# --------------------------------------------------------------------------------------------------------------
# CPU baseline: the oracle as it stands, on bounded samples of the workloads
# --------------------------------------------------------------------------------------------------------------
def cpu_baseline(sample_elems, legs=True):
    from oracle import hif8_oracle as O
    x = W.normal_f32((ROWS, COLS), seed=1234).reshape(-1)[:sample_elems]
    t0 = time.perf_counter()
    _, se = O.amax_scale(x, O.F32, 14)
    codes = O.encode(x, O.F32, se, O.TA, 0, quick=False)
    O.decode(codes, O.F32, se)
    dt = time.perf_counter() - t0
    out = {"value": 14 * sample_elems / dt / 1e9, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
           "sample": f"first {sample_elems} of {N_EL} elements: amax + brute-force TA encode + decode, {dt:.2f} s",
           "elements_per_s": sample_elems / dt}
    if not legs:
        return out
    by = {}
    # LLM-activation fake-quant (BF16, Student-t body with outlier channels), fused amax, round half away
    xb = W.llm_activation_bf16(2048, 8192, seed=2345).reshape(-1)
    t0 = time.perf_counter()
    _, se = O.amax_scale(xb, O.BF16, 14)
    O.fake_quant(xb, O.BF16, se, O.TA, 0, quick=False)
    dt = time.perf_counter() - t0
    by["bf16_activation_fake_quant_TA"] = {"elements_per_s": xb.size / dt, "GBps": 6 * xb.size / dt / 1e9, "kind": "oracle (scan of 256 codes)",
                                           "sample": f"{xb.size} of {8192 * 8192} elements, {dt:.2f} s"}
    t0 = time.perf_counter()
    O.fake_quant(xb, O.BF16, se, O.HR, 0, quick=False)
    dt = time.perf_counter() - t0
    by["bf16_activation_fake_quant_HR"] = {"elements_per_s": xb.size / dt, "GBps": 4 * xb.size / dt / 1e9, "kind": "oracle (scale given)",
                                           "sample": f"{xb.size} of {8192 * 8192} elements, {dt:.2f} s"}
    # gradient-range FP32 encode: the neighbour-pair variant, which is the one the 2^32 sweep is checked with
    g = W.loguniform_f32(1 << 24, seed=3456)
    t0 = time.perf_counter()
    O.encode(g, O.F32, 0, O.TA, 0, quick=True)
    dt = time.perf_counter() - t0
    by["loguniform_f32_encode_TA"] = {"elements_per_s": g.size / dt, "GBps": 5 * g.size / dt / 1e9,
                                      "kind": "oracle, neighbour-pair (quick) variant", "sample": f"2^24 of 2^28 elements, {dt:.2f} s"}
    # GEMM: FP64 oracle on a 128 x 128 block of outputs at K = 8192
    Aq, Wq = W.random_codes((128, 8192), seed=4567), W.random_codes((8192, 128), seed=5678)
    t0 = time.perf_counter()
    O.gemm_full(Aq, Wq, False, 0, 0)
    dt = time.perf_counter() - t0
    by["gemm_fp64"] = {"TFLOPs": 2.0 * 128 * 128 * 8192 / dt / 1e12, "kind": "oracle (FP64, sum and sum of magnitudes), extrapolated",
                       "sample": f"128 x 128 outputs of 8192 x 28672 at K = 8192, {dt:.2f} s"}
    out["by_config"] = by
    return out


# --------------------------------------------------------------------------------------------------------------
# Secondary workloads
# --------------------------------------------------------------------------------------------------------------
def extra_results(H, torch, hbm_peak, tf_peak, peak_kind, tf_sustained=None):
    """Secondary workloads (each with its own roofline fraction): BF16 fake-quant of an LLM-activation tensor,
    gradient-range FP32 encode/decode, and the HiF8-operand GEMM.  Inputs are generated on the device from a
    seeded torch generator with the same recipes as workloads/ (shapes and distributions, not the same bytes).
    Returns (detail, by_config): by_config is the compact table of the headline figure of every configuration."""
    out, table = {}, {}
    g = torch.Generator(device="cuda")
    g.manual_seed(2345)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wsb = H.hif8_workspace_bytes(H.WS_FAKE_QUANT, 0)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")

    def timed(fn, reps, repeats=MIN_REPEATS, rest_s=0.0):
        """`repeats` timed regions of `reps` calls each; median / best / worst per call.  rest_s: idle time in front of
        every region (the tensor-bound legs: a region is then a burst, like the cuBLAS burst figure it is divided by)."""
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        per_call = []
        for _ in range(repeats):
            if rest_s:
                time.sleep(rest_s)
            ev0.record()
            for r in range(reps):
                fn(r)
            ev1.record()
            torch.cuda.synchronize()
            per_call.append(ev0.elapsed_time(ev1) / reps)
        return spread(per_call)

    def hbm(stat, nbytes, **more):
        d = dict(stat, GBps=nbytes / stat["ms"] / 1e6, frac=nbytes / stat["ms"] / 1e6 / hbm_peak, **more)
        return d

    def tensor(stat, flops, **more):
        return dict(stat, TFLOPs=flops / stat["ms"] / 1e9, frac=flops / stat["ms"] / 1e9 / tf_peak, **more)

    REST = 0.3  # seconds of idle in front of every timed region of a tensor-bound leg

    def sustained(fn, flops, seconds=1.0):
        """The same call back to back for about `seconds` (under the power cap), against the sustained cuBLAS figure."""
        fn(0)
        torch.cuda.synchronize()
        ev0.record(); fn(0); ev1.record(); torch.cuda.synchronize()
        n = max(8, int(seconds * 1e3 / max(ev0.elapsed_time(ev1), 1e-3)))
        ev0.record()
        for r in range(n):
            fn(r)
        ev1.record()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1) / n
        d = {"ms": ms, "calls": n, "TFLOPs": flops / ms / 1e9}
        if tf_sustained:
            d["frac_of_sustained_peak"] = flops / ms / 1e9 / tf_sustained
        return d

    def row(name, d, bound):
        # frac: of the measured peak of the bound; frac_nominal: of 8 TB/s (HBM3e) or 2.25 PFLOP/s (dense BF16)
        nominal = d["frac"] * (tf_peak / 2250.0 if bound == "tensor" else hbm_peak / 8000.0)
        table[name] = {"ms": round(d["ms"], 5), "best_ms": round(d["best_ms"], 5), "frac": round(d["frac"], 4),
                       "frac_nominal": round(nominal, 4), "bound": bound}
        if "back_to_back" in d:  # about a second of calls in a row, against the sustained cuBLAS figure
            table[name]["back_to_back_ms"] = round(d["back_to_back"]["ms"], 5)
            if "frac_of_sustained_peak" in d["back_to_back"]:
                table[name]["frac_of_sustained_peak"] = round(d["back_to_back"]["frac_of_sustained_peak"], 4)

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
        st = timed(lambda r: gr.replay(), 5)
        ms = st["ms"] / 20
        small[str(n)] = {"us_per_encode_decode_pair": ms * 1e3, "best_us": st["best_ms"] / 20 * 1e3, "GBps": 10 * n / ms / 1e6,
                         "frac": 10 * n / ms / 1e6 / hbm_peak}
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
        st = timed(lambda r: H.hif8_fake_quant(xs[r & 1], ys[r & 1], H.BF16, n, 1, 14, mode, 0, 7, None, None, ws, wsb), 20)
        fq[name] = hbm(st, 6 * n)
        row(f"C3_fake_quant_bf16_8192x8192_{name}", fq[name], "hbm")
    st = timed(lambda r: H.hif8_fake_quant(xs[r & 1], ys[r & 1], H.BF16, n, 0, 3, H.RND_TA, 0, 0), 20)
    fq["TA_given_scale"] = hbm(st, 4 * n)
    row("C3_fake_quant_bf16_8192x8192_TA_given_scale", fq["TA_given_scale"], "hbm")
    # the same tensors to HiF8 bytes with a given scale (2 B read + 1 B written): forward (TA) and backward (HR) rounding
    cq = torch.empty(n, dtype=torch.uint8, device="cuda")
    enc = {}
    for name, mode in (("TA", H.RND_TA), ("HR", H.RND_HR)):
        st = timed(lambda r: H.hif8_encode(xs[r & 1], H.BF16, cq, n, 3, mode), 20)
        enc[name] = hbm(st, 3 * n)
        row(f"C3_encode_bf16_8192x8192_{name}", enc[name], "hbm")
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
        st = timed(lambda r: H.hif8_encode(bits, H.F32, codes, n, 0, mode), 10)
        res[name] = hbm(st, 5 * n)
        row(f"C4a_loguniform_f32_2^28_{name}", res[name], "hbm")
    st = timed(lambda r: H.hif8_decode(codes, back, H.F32, n, 0), 10)
    res["decode"] = hbm(st, 5 * n)
    row("C4a_loguniform_f32_2^28_decode", res["decode"], "hbm")
    out["loguniform_f32_2^28"] = {"bytes_per_element": 5, "calls": res, "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
    # the exhaustive FP32 sweep generates its inputs in the kernel: a write-only stream, 1 B/element (one slice of 2^28 patterns)
    sweep = {}
    for name, mode in (("TA", H.RND_TA), ("HR", H.RND_HR)):
        st = timed(lambda r: H.hif8_encode_f32_patterns((r & 15) << 28, codes, n, 0, mode), 10)
        sweep[name] = hbm(st, n)
        row(f"C4b_f32_pattern_sweep_2^28_write_only_{name}", sweep[name], "hbm")
    out["f32_pattern_sweep_2^28"] = {"bytes_per_element": 1, "modes": sweep, "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
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
    st = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, K, N, 1, 14, H.RND_TA, 0, 0, None, ch_amax, ch_se), 10)
    chan["columns_[K,N]"] = hbm(st, 5 * K * N, bytes_per_element=5, note="amax kernel (2 B) + encode kernel (2 + 1 B)")
    st = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, N, K, 0, 14, H.RND_TA, 0, 0, None, ch_amax, ch_se), 10)
    chan["rows_[N,K]"] = hbm(st, 3 * K * N, bytes_per_element=3, note="one kernel, a block per row; the second read of the row hits L1/L2")
    st = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, 2 * N, K // 2, 0, 14, H.RND_TA, 0, 0, None, ch_amax2, ch_se2), 10)
    chan["rows_[2N,K/2]"] = hbm(st, 3 * K * N, bytes_per_element=3, note="rows of 4096: two rows per block")
    st = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, N // 2, 2 * K, 0, 14, H.RND_TA, 0, 0, None, ch_amax2, ch_se2), 10)
    chan["rows_[N/2,2K]"] = hbm(st, 3 * K * N, bytes_per_element=3, note="rows of 16384: held in registers, read once")
    st = timed(lambda r: H.hif8_channel_amax_scale_encode(w, H.BF16, Wq, K, N, 1, 14, H.RND_TA, 0, 0, ch_se, None, None), 10)
    chan["columns_given_exponents"] = hbm(st, 3 * K * N, bytes_per_element=3)
    for k_, v_ in chan.items():
        row(f"channel_encode_bf16_8192x28672_{k_}", v_, "hbm")
    out["channel_scaled_encode_bf16_8192x28672"] = {"calls": chan, "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
    state = torch.empty(H.SCALE_STATE_BYTES, dtype=torch.uint8, device="cuda")
    H.hif8_scale_state_init(state, 4)
    dl = {}
    for name, measure in (("measuring_iteration", 1), ("plain_iteration", 0)):
        st = timed(lambda r: H.hif8_delayed_scale_encode(a, H.BF16, Aq, M * K, H.RND_TA, 0, 0, state, measure, 14), 20)
        dl[name] = hbm(st, 3 * M * K)
        row(f"delayed_scale_encode_bf16_8192x8192_{name}", dl[name], "hbm")
    tr = {}
    for name, mode in (("TA", H.RND_TA), ("HR", H.RND_HR)):
        st = timed(lambda r: H.hif8_encode_transpose(a, H.BF16, Aq, M, K, 3, None, mode), 20)
        tr[name] = hbm(st, 3 * M * K)
        row(f"encode_transpose_bf16_8192x8192_{name}", tr[name], "hbm")
    out["encode_transpose_bf16_8192x8192"] = {"bytes_per_element": 3, "modes": tr, "peak": hbm_peak, "peak_kind": f"of {peak_kind}"}
    out["delayed_scale_encode_bf16_8192x8192"] = {"bytes_per_element": 3, "calls": dl, "peak": hbm_peak,
                                                  "peak_kind": f"of {peak_kind}"}
    H.hif8_amax_scale_encode(a, H.BF16, Aq, M * K, 14, H.RND_TA, 0, 0, None, None, se[0:1], None, ws, wsb)
    H.hif8_amax_scale_encode(w, H.BF16, Wq, K * N, 14, H.RND_TA, 0, 0, None, None, se[1:2], None, ws, wsb)
    del a, w
    C = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    gws_b = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N)
    gws = torch.empty(gws_b, dtype=torch.uint8, device="cuda")
    flops = 2.0 * M * N * K
    f_once = lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, gws_b)
    f_fused = lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, 256)
    g_once = tensor(timed(f_once, 5, rest_s=REST), flops, device_status=H.hif8_last_device_status(),
                    note="whole call: decode of both operands to BF16 workspace + tcgen05 kernel",
                    back_to_back=sustained(f_once, flops))
    g_fused = tensor(timed(f_fused, 3, rest_s=REST), flops, device_status=H.hif8_last_device_status(),
                     note="no workspace: byte tiles decoded per CTA pair inside the tensor-core kernel",
                     back_to_back=sustained(f_fused, flops))
    gws_a = H.hif8_workspace_bytes(H.WS_GEMM, M * K)
    g_aexp = tensor(timed(lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, gws_a), 3, rest_s=REST),
                    flops, device_status=H.hif8_last_device_status(),
                    note="workspace for A alone: A expanded once to BF16, W tiles decoded inside the tensor-core kernel")
    # the same with the weight bytes read as [N,K] (the layout of a stored checkpoint; values differ, time does not depend on
    # them): the swapped form, weight rows decoded into tensor memory
    g_aexp_nk = tensor(timed(lambda r: H.hif8_gemm(Aq, K, Wq, K, 1, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, gws_a), 3, rest_s=REST),
                       flops, device_status=H.hif8_last_device_status(),
                       note="workspace for A alone, [N,K] weights: C^T = W^T A^T, weight rows decoded into tensor memory")
    ch_se.fill_(int(se[1]))
    g_chan = tensor(timed(lambda r: H.hif8_gemm_channel_scaled(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], ch_se, gws, gws_b), 5,
                          rest_s=REST),
                    flops, device_status=H.hif8_last_device_status(), note="one weight exponent per output column")
    row("C5_gemm_8192x28672x8192_decode_once", g_once, "tensor")
    row("C5_gemm_8192x28672x8192_fused", g_fused, "tensor")
    row("C5_gemm_8192x28672x8192_A_expanded_W_fused", g_aexp, "tensor")
    row("C5_gemm_8192x28672x8192_A_expanded_W_[N,K]_fused", g_aexp_nk, "tensor")
    row("gemm_8192x28672x8192_channel_scaled", g_chan, "tensor")
    # backward-pass forms of the same size: dgrad reads the weight as [N,K], wgrad reads A as [K,M] and accumulates in FP32
    bw = {}
    bw["dgrad_form_w_as_[N,K]"] = tensor(
        timed(lambda r: H.hif8_gemm_ex(Aq, K, 0, Wq, K, 1, C, N, H.BF16, M, N, K, se[0:1], se[1:2], None, 0, gws, gws_b), 5, rest_s=REST),
        flops, device_status=H.hif8_last_device_status())
    C32 = torch.zeros(M, N, dtype=torch.float32, device="cuda")
    bw["wgrad_form_a_as_[K,M]_fp32_accumulate"] = tensor(
        timed(lambda r: H.hif8_gemm_ex(Aq, M, 1, Wq, N, 0, C32, N, H.F32, M, N, K, se[0:1], se[1:2], None, 1, gws, gws_b), 5, rest_s=REST),
        flops, device_status=H.hif8_last_device_status())
    del C32
    for k_, v_ in bw.items():
        row(f"gemm_8192x28672x8192_{k_}", v_, "tensor")
    # inference-decode shapes: a few activation rows against the same weight (bound by reading the weight bytes once)
    narrow = {}
    for Mn in (16, 64):
        Cn = torch.empty(Mn, N, dtype=torch.bfloat16, device="cuda")
        # with the workspace: equal (slab, k-block) ranges per SM; with the 256-byte minimum: one CTA per slab
        byt = K * N + Mn * K + 2 * Mn * N
        st = timed(lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, Cn, N, H.BF16, Mn, N, K, se[0:1], se[1:2], gws, gws_b), 20)
        st_s = timed(lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, Cn, N, H.BF16, Mn, N, K, se[0:1], se[1:2], gws, 256), 20)
        # the same bytes read as an [N,K] weight (the layout of a stored checkpoint; values differ, time does not depend on them)
        st_nk = timed(lambda r: H.hif8_gemm(Aq, K, Wq, K, 1, Cn, N, H.BF16, Mn, N, K, se[0:1], se[1:2], gws, gws_b), 20)
        d = hbm(st, byt, us=st["ms"] * 1e3, us_one_cta_per_slab=st_s["ms"] * 1e3, us_weights_as_NK=st_nk["ms"] * 1e3,
                device_status=H.hif8_last_device_status())
        d["frac_of_hbm"] = d["frac"]
        narrow[f"M={Mn}"] = d
        row(f"gemm_narrow_{Mn}x28672x8192", d, "hbm (weight bytes)")
        row(f"gemm_narrow_{Mn}x28672x8192_weights_as_[N,K]", hbm(st_nk, byt), "hbm (weight bytes)")
        del Cn
    # prefill-sized products against the same weight, with the full workspace: below about 1600 rows the call expands A alone
    mid = {}
    for Mm in (256, 1024):
        Cm = torch.empty(Mm, N, dtype=torch.bfloat16, device="cuda")
        stm = timed(lambda r: H.hif8_gemm(Aq, K, Wq, N, 0, Cm, N, H.BF16, Mm, N, K, se[0:1], se[1:2], gws, gws_b), 10, rest_s=REST)
        mid[f"M={Mm}"] = tensor(stm, 2.0 * Mm * N * K, us=stm["ms"] * 1e3, device_status=H.hif8_last_device_status())
        row(f"gemm_{Mm}x28672x8192_full_workspace", mid[f"M={Mm}"], "tensor")
        del Cm
    out["gemm_midM_x28672x8192"] = {"bound": "tensor", "shapes": mid, "peak": tf_peak, "peak_kind": f"of {peak_kind} (cuBLAS BF16 burst)",
                                    "note": "the weight bytes alone take 36 us at the copy rate; 256 rows run as one tile row of 256"}
    out["gemm_narrow_Mx28672x8192"] = {"bound": "hbm", "bytes": "K*N weight bytes + M*K + 2*M*N", "shapes": narrow,
                                       "peak": hbm_peak, "peak_kind": f"of {peak_kind}",
                                       "note": "whole call; with the workspace it first expands the activations to BF16 (one more launch, "
                                               "2*M*K bytes) and splits the weight evenly over the SMs"}
    out["gemm_8192x28672x8192"] = {
        "backward_forms": bw, "decode_once_channel_scaled": g_chan, "decode_once": g_once, "fused": g_fused, "a_expanded_w_fused": g_aexp, "a_expanded_w_nk_fused": g_aexp_nk,
        "bound": "tensor", "peak": tf_peak, "peak_kind": f"of {peak_kind} (cuBLAS BF16 burst)", "unit": "TFLOP/s",
        "timing": f"every timed region starts after {REST} s of idle (bursts, like the peak); back_to_back: about one second of calls "
                  "in a row under the power cap, against the sustained cuBLAS figure",
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
    st = timed(lambda r: H.hif8_pts_search(a, w, H.BF16, 0, o_ref, N, M, N, K, -4, 5, d_err, d_best, pws, pb), 2, repeats=3)
    pts = tensor(st, 100 * 2.0 * M * N * K, best_exponents=[int(v) for v in d_best.cpu()], device_status=H.hif8_pts_status(pws),
                 min_mse=float(d_err.min().item()))
    pts["TFLOPs_of_100_gemms"] = pts["TFLOPs"]
    out["pts_search_4096^3"] = pts
    row("algorithm1_search_4096^3_10x10", pts, "tensor")
    return out, table


# --------------------------------------------------------------------------------------------------------------
# Named workloads for a profiler (a few launches each; nothing is timed or printed but a completion line)
# --------------------------------------------------------------------------------------------------------------
CASES = ("convert_f32", "fq_bf16", "encode_modes_f32", "encode_modes_bf16", "transpose_bf16", "gemm", "gemm_fused", "gemm_narrow",
         "gemm_forms", "gemm_a_expanded", "channel_bf16")


def run_case(case, reps):
    """convert_f32: FP32 4096^2 per-tensor scaled encode + decode over three rotating tensors (the bench step);
    fq_bf16: BF16 4096x8192 fake-quant, TA / HR / TE, fused amax and given scale; encode_modes_f32 / encode_modes_bf16:
    2^25 log-uniform values in every rounding mode; transpose_bf16: BF16 8192^2 flat and transposed-store encode, TA and
    HR; gemm: HiF8 GEMM 4096 x 7168 x 4096 on the decode-once and the fused path (gemm_fused: the fused path only);
    gemm_forms: the four operand layouts on the decode-once path; gemm_a_expanded: the same size with a workspace for A alone, [K,N] and [N,K] weights;
    gemm_narrow: 16 x 8192 x 8192 with weights as [K,N] and
    [N,K] (equal ranges of the weight per SM); channel_bf16: per-channel scaled encode of a BF16 8192 x 14336 weight by column and by row, plus the overflow
    check.  Inputs are seeded device-side random tensors."""
    import torch
    import paper_2409_16626_b200 as H
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    if case in ("gemm", "gemm_forms"):  # these cases exist to capture the decode-once kernel: ask for it whatever the size
        H.hif8_gemm_path_policy(H.GEMM_PATH_EXPAND_BOTH)
    if case == "convert_f32":
        n = N_EL
        xs = [torch.randn(n, generator=g, device="cuda") for _ in range(3)]
        codes = torch.empty(n, dtype=torch.uint8, device="cuda")
        back = torch.empty(n, dtype=torch.float32, device="cuda")
        se = torch.zeros(1, dtype=torch.int32, device="cuda")
        for r in range(reps):
            H.hif8_amax_scale_encode(xs[r % 3], H.F32, codes, n, 14, H.RND_TA, 0, 0, None, None, se, None, ws, 256)
            H.hif8_decode(codes, back, H.F32, n, 12)
    elif case == "fq_bf16":
        n = 4096 * 8192
        xs = [torch.randn(n, generator=g, device="cuda").to(torch.bfloat16) for _ in range(3)]
        y = torch.empty_like(xs[0])
        for r in range(reps):
            for mode in (H.RND_TA, H.RND_HR, H.RND_TE):
                H.hif8_fake_quant(xs[r % 3], y, H.BF16, n, 1, 14, mode, 0, 7, None, None, ws, 256)
                H.hif8_fake_quant(xs[r % 3], y, H.BF16, n, 0, 12, mode, 0, 7)
    elif case in ("encode_modes_f32", "encode_modes_bf16"):
        n = 1 << 25
        f32 = case == "encode_modes_f32"
        e = torch.randint(-40, 20, (n,), generator=g, device="cuda", dtype=torch.int32) + 127
        m = torch.randint(0, 1 << (23 if f32 else 7), (n,), generator=g, device="cuda", dtype=torch.int32)
        bits = (e << 23) | m if f32 else ((e << 7) | m).to(torch.int16)
        codes = torch.empty(n, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            for mode in (H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR):
                H.hif8_encode(bits, H.F32 if f32 else H.BF16, codes, n, 0, mode, 0, 5)
    elif case == "transpose_bf16":
        R, Cc = 8192, 8192
        xs = [torch.randn(R * Cc, generator=g, device="cuda").to(torch.bfloat16) for _ in range(2)]
        codes = torch.empty(R * Cc, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            for mode in (H.RND_TA, H.RND_HR):
                H.hif8_encode(xs[r & 1], H.BF16, codes, R * Cc, 3, mode, 0, 5)
                H.hif8_encode_transpose(xs[r & 1], H.BF16, codes, R, Cc, 3, None, mode)
    elif case in ("gemm", "gemm_fused"):
        M, N, K = 4096, 7168, 4096
        A = torch.randint(0, 256, (M, K), dtype=torch.uint8, device="cuda", generator=g)
        Wt = torch.randint(0, 256, (K, N), dtype=torch.uint8, device="cuda", generator=g)
        for t in (A, Wt):                                  # keep the operands finite
            t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x08
        C = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        big = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N)
        gws = torch.empty(big, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            if case == "gemm":
                H.hif8_gemm(A, K, Wt, N, 0, C, N, H.BF16, M, N, K, None, None, gws, big)
            H.hif8_gemm(A, K, Wt, N, 0, C, N, H.BF16, M, N, K, None, None, gws, 256)
    elif case == "gemm_narrow":
        M, N, K = 16, 8192, 8192
        A = torch.randint(8, 100, (M * K,), dtype=torch.uint8, device="cuda", generator=g)
        Wt = torch.randint(8, 100, (K * N,), dtype=torch.uint8, device="cuda", generator=g)
        C = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
        big = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N)
        gws = torch.empty(big, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            H.hif8_gemm(A, K, Wt, N, 0, C, N, H.BF16, M, N, K, None, None, gws, big)
            H.hif8_gemm(A, K, Wt, K, 1, C, N, H.BF16, M, N, K, None, None, gws, big)
    elif case == "gemm_a_expanded":
        M, N, K = 4096, 7168, 4096
        A = torch.randint(8, 100, (M * K,), dtype=torch.uint8, device="cuda", generator=g)
        Wt = torch.randint(8, 100, (K * N,), dtype=torch.uint8, device="cuda", generator=g)
        C = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
        a_only = H.hif8_workspace_bytes(H.WS_GEMM, M * K)
        gws = torch.empty(a_only, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            H.hif8_gemm(A, K, Wt, N, 0, C, N, H.BF16, M, N, K, None, None, gws, a_only)   # [K,N] weights
            H.hif8_gemm(A, K, Wt, K, 1, C, N, H.BF16, M, N, K, None, None, gws, a_only)   # [N,K] weights: the swapped form
    elif case == "gemm_forms":
        M, N, K = 4096, 7168, 4096
        A = torch.randint(8, 100, (M * K,), dtype=torch.uint8, device="cuda", generator=g)
        Wt = torch.randint(8, 100, (K * N,), dtype=torch.uint8, device="cuda", generator=g)
        Cb = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
        Cf = torch.zeros(M, N, dtype=torch.float32, device="cuda")
        big = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N)
        gws = torch.empty(big, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            H.hif8_gemm_ex(A, K, 0, Wt, N, 0, Cb, N, H.BF16, M, N, K, None, None, None, 0, gws, big)
            H.hif8_gemm_ex(A, K, 0, Wt, K, 1, Cb, N, H.BF16, M, N, K, None, None, None, 0, gws, big)
            H.hif8_gemm_ex(A, M, 1, Wt, N, 0, Cf, N, H.F32, M, N, K, None, None, None, 1, gws, big)
            H.hif8_gemm_ex(A, M, 1, Wt, K, 1, Cb, N, H.BF16, M, N, K, None, None, None, 0, gws, big)
    elif case == "channel_bf16":
        K, N = 8192, 14336
        w = (torch.randn(K, N, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
        q = torch.empty(K * N, dtype=torch.uint8, device="cuda")
        amax = torch.empty(N, dtype=torch.float32, device="cuda")
        se = torch.empty(N, dtype=torch.int32, device="cuda")
        flag = torch.zeros(1, dtype=torch.int32, device="cuda")
        for r in range(reps):
            H.hif8_channel_amax_scale_encode(w, H.BF16, q, K, N, 1, 14, H.RND_TA, 0, 0, None, amax, se)
            H.hif8_channel_amax_scale_encode(w, H.BF16, q, N, K, 0, 14, H.RND_TA, 0, 0, None, amax, se)
            H.hif8_check_finite(w, H.BF16, K * N, flag)
    else:
        raise SystemExit(f"unknown case {case}; one of {', '.join(CASES)}")
    torch.cuda.synchronize()
    print("done", case, H.hif8_launch_count())


# --------------------------------------------------------------------------------------------------------------
# Reference arm: the CPU oracle
# --------------------------------------------------------------------------------------------------------------
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


# --------------------------------------------------------------------------------------------------------------
# Multi-GPU figures beside the headline (world > 1): a tensor sharded over the ranks, and the column-sharded GEMM
# --------------------------------------------------------------------------------------------------------------
def sharded_results(H, torch, dist, rank, world, stream):
    from paper_2409_16626_b200 import sharded
    out = {}
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps):
        for _ in range(3):
            fn()
        dist.barrier()
        torch.cuda.synchronize()
        ev0.record(stream)
        for _ in range(reps):
            fn()
        ev1.record(stream)
        torch.cuda.synchronize()
        dist.barrier()
        return max_over_ranks([ev0.elapsed_time(ev1) / reps], dist, "cuda")[0]

    # the 4096 x 4096 FP32 tensor split into `world` contiguous slices: hif8_amax -> 4-byte max all-reduce (NCCL) ->
    # hif8_encode_from_amax; 9 algorithmic bytes per element as for the just-in-time call on one GPU
    lo, hi = sharded.shard_range(N_EL, world, rank, 16)
    shard = torch.from_numpy(W.normal_f32((ROWS, COLS), seed=1234).reshape(-1)[lo:hi].copy()).cuda()
    dst = torch.empty(hi - lo, dtype=torch.uint8, device="cuda")
    d_amax = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    ms = timed(lambda: sharded.sharded_amax_scale_encode(H, shard, H.F32, dst, hi - lo, 14, H.RND_TA, 0, 0, d_amax, ws, 256), 50)
    out["sharded_amax_scale_encode_fp32_4096x4096"] = {"ms": ms, "GBps_whole_tensor": 9 * N_EL / ms / 1e6, "scaling": "strong",
                                                       "collective": "one 4-byte max all-reduce (NCCL)"}
    # GEMM 8192 x 28672 x 8192 with Wq split along N: every rank multiplies the whole A by its own column block and owns
    # that block of C; no collective on the data path
    M, N, K = 8192, 28672, 8192
    c0, c1 = sharded.shard_range(N, world, rank, 256)
    g = torch.Generator(device="cuda")
    g.manual_seed(77)
    Aq = torch.randint(8, 100, (M, K), dtype=torch.uint8, device="cuda", generator=g)
    Wq = torch.randint(8, 100, (K, c1 - c0), dtype=torch.uint8, device="cuda", generator=g)
    C = torch.empty(M, c1 - c0, dtype=torch.bfloat16, device="cuda")
    gb = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * (c1 - c0))
    gws = torch.empty(gb, dtype=torch.uint8, device="cuda")
    ms = timed(lambda: sharded.column_sharded_gemm(H, Aq, Wq, C, M, c1 - c0, K, None, None, gws, gb), 3)
    out["gemm_8192x28672x8192_w_sharded_along_n"] = {"ms": ms, "TFLOPs_whole_job": 2.0 * M * N * K / ms / 1e9, "scaling": "strong",
                                                     "collective": "none", "columns_of_rank0": [c0, c1]}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the secondary workloads (fake-quant, 2^28 stress, GEMM)")
    ap.add_argument("--case", default=None, help="run one named workload a few times and exit (for a profiler): " + ", ".join(CASES))
    ap.add_argument("--reps", type=int, default=3, help="repetitions of --case")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    rank, world, local = env_int("RANK", 0), env_int("WORLD_SIZE", 1), env_int("LOCAL_RANK", 0)

    if args.case:
        run_case(args.case, args.reps)
        return
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

    H.hif8_amax_scale_encode(srcs[0], H.F32, codes[0], N_EL, 14, H.RND_TA, 0, 0, None, scal[0:1], scal[1:2], scal[2:3], ws, wsb, stream=sp)
    torch.cuda.synchronize()
    se = int(scal[1].item())   # same distribution for every tensor of the pool: the descale exponent is fixed up front
    d_se = scal[1:2].clone()

    for w in range(args.warmup):
        H.hif8_amax_scale_encode(srcs[w % POOL], H.F32, codes[w % POOL], N_EL, 14, H.RND_TA, 0, 0, None, scal[0:1], scal[1:2],
                                 scal[2:3], ws, wsb, stream=sp)
        H.hif8_decode(codes[w % POOL], backs[w % POOL], H.F32, N_EL, se, stream=sp)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: device-resident inputs, CUDA events on the launching stream.
    # The launch sequence of POOL consecutive steps (one per buffer set) is captured once in a CUDA graph and
    # replayed, so the host's per-launch cost stays out of the device timeline; K steps = K // POOL replays of that
    # graph plus one replay of a second graph holding the remaining K % POOL steps, so exactly K steps are timed.
    # The region of K steps is repeated (at least MIN_REPEATS times, more when it is short) and the median region is the
    # one reported, with the best and the worst beside it.
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

    def time_region(gr, tail, repeats):
        """per-step times (ms) of `repeats` regions of exactly K steps each; max over ranks per region"""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        per_step = []
        for _ in range(repeats):
            barrier()
            a.record(stream)
            replay_steps(gr, tail)
            b.record(stream)
            torch.cuda.synchronize()
            per_step.append(a.elapsed_time(b) / K)
        barrier()
        return max_over_ranks(per_step, dist if world > 1 else None, "cuda")

    def warm(gr, tail):
        for _ in range(W_REPLAYS):
            gr.replay()
        if tail is not None:
            tail.replay()
        torch.cuda.synchronize()

    serial, serial_tail = capture(False), (capture(False, K % POOL) if K % POOL else None)
    graph, graph_tail = capture(True), (capture(True, K % POOL) if K % POOL else None)
    warm(serial, serial_tail)
    warm(graph, graph_tail)
    R = repeats_for(K * 0.035)

    def kernel_stats(call):
        """one call of the step in a graph of its own (POOL launches over the rotating buffers), replayed between two
        events: direct launches would time the host's launch rate, not these ~15 us kernels"""
        gk = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gk):
            cs = torch.cuda.current_stream().cuda_stream
            for i in range(POOL):
                call(i, cs)
        reps = max(4, min(K, 600) // POOL)
        for _ in range(3):
            gk.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        per = []
        for _ in range(MIN_REPEATS):
            a.record(stream)
            for _ in range(reps):
                gk.replay()
            b.record(stream)
            torch.cuda.synchronize()
            per.append(a.elapsed_time(b) / (reps * POOL))
        return per

    amax_out = torch.zeros(1, dtype=torch.float32, device="cuda")
    with ClockSampler(local) as clk:
        step_samples = time_region(graph, graph_tail, R)
        serial_samples = time_region(serial, serial_tail, R)
        k_amax = kernel_stats(lambda i, cs: H.hif8_amax(srcs[i], H.F32, N_EL, amax_out, ws, wsb, stream=cs))
        k_conv = kernel_stats(lambda i, cs: H.hif8_encode(srcs[i], H.F32, codes[i], N_EL, se, H.RND_TA, 0, 0, stream=cs))
        k_dec = kernel_stats(lambda i, cs: H.hif8_decode(codes[i], backs[i], H.F32, N_EL, se, stream=cs))
        k_enc = kernel_stats(lambda i, cs: H.hif8_amax_scale_encode(srcs[i], H.F32, codes[i], N_EL, 14, H.RND_TA, 0, 0, None,
                                                                    scal[0:1], scal[1:2], scal[2:3], ws, wsb, stream=cs))
        # delayed-scaling form of the same conversion: the exponent comes from device memory, amax of this tensor is
        # reduced in the same pass (one launch, 5 B/element)
        k_del = kernel_stats(lambda i, cs: H.hif8_amax_scale_encode(srcs[i], H.F32, codes[i], N_EL, 14, H.RND_TA, 0, 0, d_se,
                                                                    scal[0:1], None, None, ws, wsb, stream=cs))
    launches = 4 * K   # accumulator clear + amax + convert + decode kernels per step (graph replays), per timed region

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
    e2e_ms = max_over_ranks([e0.elapsed_time(e1) / E], dist if world > 1 else None, "cuda")[0]
    if world > 1:
        k_amax, k_conv, k_dec, k_enc, k_del = [max_over_ranks(v, dist, "cuda") for v in (k_amax, k_conv, k_dec, k_enc, k_del)]
        try:   # secondary figures: a failure here must not take the headline line with it
            multi = sharded_results(H, torch, dist, rank, world, stream)
        except Exception as exc:  # noqa: BLE001
            multi = {"error": f"{type(exc).__name__}: {exc}"}

    if rank == 0:
        step, serial_st = spread(step_samples), spread(serial_samples)
        ms_per_step = step["ms"]
        value = job_throughput(world, BYTES_STEP, ms_per_step)
        peak, tf_peak, tf_sustained, peak_kind = load_peaks()
        kernels = {
            "amax_kernel<f32>": dict(spread(k_amax), bytes=4 * N_EL, note="hif8_amax call: accumulator-clearing kernel + amax kernel"),
            "convert_kernel<f32,TA>": dict(spread(k_conv), bytes=5 * N_EL),
            "decode_kernel<f32>": dict(spread(k_dec), bytes=5 * N_EL),
        }
        for kv in kernels.values():
            kv["GBps"] = kv["bytes"] / (kv["ms"] * 1e-3) / 1e9
            kv["frac"] = kv["GBps"] / peak
        enc_st, del_st = spread(k_enc), spread(k_del)
        # the dominant kernel: longest live duration among the single-kernel calls
        dom = max(("convert_kernel<f32,TA>", "decode_kernel<f32>"), key=lambda kname: kernels[kname]["ms"])

        def row(st, nbytes):
            return {"ms": round(st["ms"], 5), "best_ms": round(st["best_ms"], 5), "frac": round(nbytes / st["ms"] / 1e6 / peak, 4),
                    "frac_nominal": round(nbytes / st["ms"] / 1e6 / 8000.0, 4), "bound": "hbm"}

        by_config = {
            "C2_step_two_streams_14B_per_el_algorithmic": row(step, BYTES_STEP),
            "C2_step_single_stream_14B_per_el_algorithmic": row(serial_st, BYTES_STEP),
            "C2_amax_scale_encode_call_9B_per_el": row(enc_st, BYTES_ENCODE),
            "C2_delayed_scaling_encode_call_5B_per_el": row(del_st, 5 * N_EL),
            "C2_amax_call_4B_per_el": row(kernels["amax_kernel<f32>"], 4 * N_EL),
            "C2_convert_kernel_5B_per_el": row(kernels["convert_kernel<f32,TA>"], 5 * N_EL),
            "C2_decode_kernel_5B_per_el": row(kernels["decode_kernel<f32>"], 5 * N_EL),
        }
        in_step = [TRAFFIC_IN_STEP[k] for k in ("amax_kernel<f32>", "convert_kernel<f32,TA>", "decode_kernel<f32>")]
        dram_step = sum(in_step) if all(v is not None for v in in_step) else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "elements": N_EL, "rounding": "TA", "target_exp": 14,
                       "value_is": "algorithmic bytes per second (14 B/element: both reads of the source and the read of the "
                                   "codes are counted although the L2 can serve them), not a DRAM bandwidth",
                       "launch": f"CUDA graph of {POOL} steps replayed (+ one graph of steps % {POOL}); even/odd steps "
                                 "(independent tensors) on two streams",
                       "timed": f"{step['repeats']} regions of exactly {K} steps each; ms_per_step is the median region",
                       "ms_per_step_best": step["best_ms"], "ms_per_step_worst": step["worst_ms"],
                       "ms_per_step_single_stream": serial_st["ms"], "ms_per_step_single_stream_best": serial_st["best_ms"],
                       "GBps_single_stream": job_throughput(world, BYTES_STEP, serial_st["ms"]),
                       "step_dram": {"bytes_per_step": dram_step,
                                     "GBps": None if dram_step is None else world * dram_step / (ms_per_step * 1e-3) / 1e9,
                                     "frac_of_peak": None if dram_step is None else dram_step / (ms_per_step * 1e-3) / 1e9 / peak,
                                     "source": "dram__bytes_read.sum + dram__bytes_write.sum of the three kernels inside the running "
                                               "sequence (profiler capture with the caches left alone between launches)"},
                       "l2": f"inputs rotate over {POOL} buffer sets ({POOL * N_EL * 4 >> 20} MiB of sources) > 126 MB L2",
                       "bytes_per_step": BYTES_STEP, "elements_per_s": world * N_EL / (ms_per_step * 1e-3)},
            "clocks": clk.summary(),
            "e2e": {"value": job_throughput(world, BYTES_STEP, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": 4 * N_EL, "d2h_bytes_per_step": 5 * N_EL},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["GBps"], "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": kernels[dom]["frac"],
                         "traffic": TRAFFIC_COLD.get(dom), "traffic_in_step": TRAFFIC_IN_STEP.get(dom),
                         "algorithmic_bytes_per_launch": kernels[dom]["bytes"],
                         "avg_launch_ms": kernels[dom]["ms"], "best_launch_ms": kernels[dom]["best_ms"],
                         "by_config": by_config,
                         "by_config_peaks": {"hbm": peak, "tensor": tf_peak, "tensor_sustained": tf_sustained, "kind": f"of {peak_kind}",
                                             "units": "frac = algorithmic GB/s / hbm, or TFLOP/s / tensor (cuBLAS BF16 burst); frac_nominal: of 8000 GB/s or 2250 TFLOP/s"}},
            "kernels": kernels,
            "calls": {"amax_scale_encode_ms": enc_st["ms"], "amax_scale_encode_GBps": BYTES_ENCODE / (enc_st["ms"] * 1e-3) / 1e9,
                      "delayed_scaling_encode_ms": del_st["ms"]},
        }
        if world > 1:
            line["sharded"] = multi
        if world == 1 and not args.no_extra:
            del srcs, codes, backs
            torch.cuda.empty_cache()
            line["extra"], table = extra_results(H, torch, peak, tf_peak, peak_kind, tf_sustained)
            by_config.update(table)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(1 << 23)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
