"""Parity at the full workload sizes, in the launch configuration bench.py times, on sampled outputs.

Inputs are generated on the device from a seeded torch generator (same recipes as workloads/); the sampled
elements are copied back and go through the CPU oracle one by one.
"""
import numpy as np
import pytest
import torch

import paper_2409_16626_b200 as H
from oracle import hif8_oracle as O

pytestmark = pytest.mark.gpu


def _gen(seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return g


def _sample_idx(n, count, seed):
    rng = np.random.default_rng(seed)
    idx = np.unique(np.concatenate([rng.integers(0, n, count), np.arange(0, 40000), np.arange(n - 40000, n)]))
    return idx


def test_config3_bf16_activation_fake_quant_all_modes():
    # BF16 [8192 x 8192]: Student-t(3) body, 0.1 % of hidden channels x100; fused amax + quantize-dequantize
    T = Hd = 8192
    n = T * Hd
    g = _gen(2345)
    z = torch.randn(T, Hd, generator=g, device="cuda")
    chi = torch.zeros_like(z)
    for _ in range(3):
        chi += torch.randn(T, Hd, generator=g, device="cuda") ** 2
    x = z / torch.sqrt(chi / 3.0)
    cols = torch.randperm(Hd, generator=g, device="cuda")[:8]
    x[:, cols] *= 100.0
    xb = x.to(torch.bfloat16).reshape(-1)
    del z, chi, x
    y = torch.empty_like(xb)
    wsb = H.hif8_workspace_bytes(H.WS_FAKE_QUANT, n)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    outs = torch.zeros(2, dtype=torch.int32, device="cuda")
    idx = _sample_idx(n, 400_000, 1)
    tidx = torch.from_numpy(idx).cuda()
    src_s = xb.view(torch.int16)[tidx].cpu().numpy().view(np.uint16)
    amax_ref = float(xb.float().abs().max().item())             # library reduction, only to cross-check amax
    for mode in (H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR):
        H.hif8_fake_quant(xb, y, H.BF16, n, 1, 14, mode, 0, 77, outs[0:1], outs[1:2], ws, wsb)
        torch.cuda.synchronize()
        o = outs.cpu().numpy()
        assert o[0:1].view(np.float32)[0] == np.float32(amax_ref)
        se = int(o[1])
        assert 2.0 ** 14 <= amax_ref * 2.0 ** se < 2.0 ** 15
        got = y.view(torch.int16)[tidx].cpu().numpy().view(np.uint16)
        if mode == H.RND_SR:
            # the threshold of element i depends on i: check the leading 40,000 elements (their positions are their
            # indices), and that every other sampled output is one of the two neighbouring HiF8 values
            head = xb.view(torch.int16)[:40000].cpu().numpy().view(np.uint16)
            want = O.fake_quant(head, O.BF16, se, O.SR, 0, seed=77, quick=True)
            assert np.array_equal(y.view(torch.int16)[:40000].cpu().numpy().view(np.uint16), want)
            lo = O.fake_quant(src_s, O.BF16, se, O.SSR, 0, quick=True)       # one neighbour ...
            ta = O.fake_quant(src_s, O.BF16, se, O.TA, 0, quick=True)        # ... or the nearest one
            gv, lv, tv = [v.astype(np.uint32) << 16 for v in (got, lo, ta)]
            gf, lf, tf = [v.view(np.float32).astype(np.float64) for v in (gv, lv, tv)]
            fin = np.isfinite(tf) & np.isfinite(lf) & np.isfinite(gf)
            span = np.maximum(np.abs(lf - tf), np.abs(tf) * 2.0 ** -1)      # at most one HiF8 step away from TA
            assert np.all(np.abs(gf - tf)[fin] <= span[fin] + 1e-300)
        else:
            want = O.fake_quant(src_s, O.BF16, se, mode, 0, seed=77, quick=True)
            assert np.array_equal(got, want), f"mode {mode}: {np.count_nonzero(got != want)} mismatches"


def test_config4a_gradient_range_fp32_2_28():
    # FP32, 2^28 elements, log-uniform magnitudes over 2^-40 .. 2^20, random signs, unscaled; TA and HR; decode
    n = 1 << 28
    g = _gen(3456)
    e = torch.randint(-40, 20, (n,), generator=g, device="cuda", dtype=torch.int32) + 127
    m = torch.randint(0, 1 << 23, (n,), generator=g, device="cuda", dtype=torch.int32)
    sg = torch.randint(0, 2, (n,), generator=g, device="cuda", dtype=torch.int32)
    bits = (sg << 31) | (e << 23) | m
    del e, m, sg
    codes = torch.empty(n, dtype=torch.uint8, device="cuda")
    idx = _sample_idx(n, 1_000_000, 2)
    tidx = torch.from_numpy(idx).cuda()
    src_s = bits[tidx].cpu().numpy().view(np.uint32)
    for mode in (H.RND_TA, H.RND_HR):
        H.hif8_encode(bits, H.F32, codes, n, 0, mode)
        torch.cuda.synchronize()
        got = codes[tidx].cpu().numpy()
        want = O.encode(src_s, O.F32, 0, mode, 0, quick=True)
        assert np.array_equal(got, want), f"mode {mode}: {np.count_nonzero(got != want)} mismatches"
    # underflow to the single zero, the denormal extension and overflow all occur in the sample
    assert (want == 0).any() and ((want & 0x7F) < 8).any() and ((want & 0x7F) == 0x6F).any()
    back = torch.empty(n, dtype=torch.float32, device="cuda")
    H.hif8_decode(codes, back, H.F32, n, 0)
    torch.cuda.synchronize()
    assert np.array_equal(back[tidx].cpu().numpy().view(np.uint32), O.decode(got, O.F32, 0))


@pytest.mark.parametrize("staged", [True, False])
def test_config5_gemm_8192x28672x8192(staged):
    # A BF16 8192 x 8192 N(0,1), W BF16 8192 x 28672 N(0,0.02): per-tensor scaled, encoded, multiplied; BF16 out
    M, N, K = 8192, 28672, 8192
    g = _gen(4567)
    a = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
    w = (torch.randn(K, N, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    Aq = torch.empty(M * K, dtype=torch.uint8, device="cuda")
    Wq = torch.empty(K * N, dtype=torch.uint8, device="cuda")
    se = torch.zeros(2, dtype=torch.int32, device="cuda")
    wsb = H.hif8_workspace_bytes(H.WS_AMAX_SCALE_ENCODE, 0)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    H.hif8_amax_scale_encode(a, H.BF16, Aq, M * K, 14, H.RND_TA, 0, 0, None, None, se[0:1], None, ws, wsb)
    H.hif8_amax_scale_encode(w, H.BF16, Wq, K * N, 14, H.RND_TA, 0, 0, None, None, se[1:2], None, ws, wsb)
    del a, w
    C = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    gb = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N) if staged else H.hif8_workspace_bytes(H.WS_GEMM, 0)
    gws = torch.empty(gb, dtype=torch.uint8, device="cuda")
    H.hif8_gemm(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, gb)
    assert H.hif8_gemm_status(gws) == 0
    sa, sw = [int(v) for v in se.cpu()]
    rng = np.random.default_rng(3)
    rows = np.concatenate([rng.integers(0, M, 60000), np.repeat(np.arange(M - 128, M), 256), np.repeat(np.arange(4096, 4096 + 64), 256)])
    cols = np.concatenate([rng.integers(0, N, 60000), np.tile(np.arange(N - 256, N), 128), np.tile(np.arange(14336 - 128, 14336 + 128), 64)])
    Cs, S = O.gemm_entries(Aq.cpu().numpy().reshape(M, K), Wq.cpu().numpy().reshape(K, N), False, sa, sw, rows, cols)
    got = C[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()].float().cpu().numpy().astype(np.float64)
    tol = 1e-5 * S + 2.0 ** -8 * np.abs(Cs)
    err = np.abs(got - Cs)
    assert np.all(err <= tol), f"{np.count_nonzero(err > tol)} outside tolerance, worst ratio {np.max(err / tol):.3g}"
