"""Parity at the full workload sizes, in the launch configuration bench.py times.

Inputs are generated on the device from a seeded torch generator (same recipes as workloads/).  The conversion
workloads are compared in full, element by element, with the oracle's neighbour-pair variant (cross-checked against
the 256-code scan in the oracle's own pins, and here on a sample); the GEMM on sampled outputs.
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
    src_all = xb.view(torch.int16).cpu().numpy().view(np.uint16)
    amax_ref, se_ref = O.amax_scale(src_all, O.BF16, 14)
    for mode in (H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR):
        H.hif8_fake_quant(xb, y, H.BF16, n, 1, 14, mode, 0, 77, outs[0:1], outs[1:2], ws, wsb)
        torch.cuda.synchronize()
        o = outs.cpu().numpy()
        assert o[0:1].view(np.float32)[0] == np.float32(amax_ref)
        se = int(o[1])
        assert se == se_ref and 2.0 ** 14 <= amax_ref * 2.0 ** se < 2.0 ** 15
        got = y.view(torch.int16).cpu().numpy().view(np.uint16)
        # the whole tensor; standard SR takes the word of each element's flat index (Philox blocks up to 2^24)
        want = O.fake_quant(src_all, O.BF16, se, mode, 0, seed=77, quick=True)
        assert np.array_equal(got, want), f"mode {mode}: {np.count_nonzero(got != want)} mismatches"
        # and the sampled elements through the oracle's scan of all 256 codes / its index-addressed entry
        want_s = O.fake_quant_at(src_all[idx], O.BF16, idx, se, mode, 0, seed=77, quick=False)
        assert np.array_equal(got[idx], want_s)


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
    src_all = bits.cpu().numpy().view(np.uint32)
    for mode in (H.RND_TA, H.RND_HR):
        H.hif8_encode(bits, H.F32, codes, n, 0, mode)
        torch.cuda.synchronize()
        got = codes.cpu().numpy()
        want = O.encode(src_all, O.F32, 0, mode, 0, quick=True)          # all 2^28 elements
        assert np.array_equal(got, want), f"mode {mode}: {np.count_nonzero(got != want)} mismatches"
    # underflow to the single zero, the denormal extension and overflow all occur
    assert (want == 0).any() and ((want & 0x7F) < 8).any() and ((want & 0x7F) == 0x6F).any()
    back = torch.empty(n, dtype=torch.float32, device="cuda")
    H.hif8_decode(codes, back, H.F32, n, 0)
    torch.cuda.synchronize()
    assert np.array_equal(back.cpu().numpy().view(np.uint32), O.decode(got, O.F32, 0))
    del back
    # standard SR on the same tensor: sampled elements, each with the Philox word of its own flat index (counters up
    # to 2^26, far beyond what the small cases reach), plus the head and the tail of the tensor
    H.hif8_encode(bits, H.F32, codes, n, 0, H.RND_SR, 0, 4242)
    torch.cuda.synchronize()
    idx = _sample_idx(n, 1_000_000, 2)
    got = codes[torch.from_numpy(idx).cuda()].cpu().numpy()
    want = O.encode_at(src_all[idx], O.F32, idx, 0, O.SR, 0, seed=4242, quick=True)
    assert np.array_equal(got, want), f"SR: {np.count_nonzero(got != want)} mismatches"


@pytest.mark.parametrize("staged", [True, False, "a", "a_nk"])  # "a": workspace for A alone; "a_nk": the same with [N,K] weights
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
    gb = H.hif8_workspace_bytes(H.WS_GEMM, (M * K + K * N) if staged is True else (M * K if staged else 0))
    gws = torch.empty(gb, dtype=torch.uint8, device="cuda")
    if staged == "a_nk":
        Wt = Wq.view(K, N).t().contiguous().view(-1)
        H.hif8_gemm(Aq, K, Wt, K, 1, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, gb)
        del Wt
    else:
        H.hif8_gemm(Aq, K, Wq, N, 0, C, N, H.BF16, M, N, K, se[0:1], se[1:2], gws, gb)
    assert H.hif8_gemm_status(gws) == 0
    sa, sw = [int(v) for v in se.cpu()]
    rng = np.random.default_rng(3)
    rows = np.concatenate([rng.integers(0, M, 60000), np.repeat(np.arange(M - 128, M), 256), np.repeat(np.arange(4096, 4096 + 64), 256)])
    cols = np.concatenate([rng.integers(0, N, 60000), np.tile(np.arange(N - 256, N), 128), np.tile(np.arange(14336 - 128, 14336 + 128), 64)])
    Cs, S = O.gemm_entries(Aq.cpu().numpy().reshape(M, K), Wq.cpu().numpy().reshape(K, N), False, sa, sw, rows, cols)
    got = C[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()].float().cpu().numpy().astype(np.float64)
    tol = 1e-5 * S
    tol = tol + 2.0 ** (np.floor(np.log2(np.maximum(np.abs(Cs) + tol, 2.0 ** -126))) - 8)   # + half a BF16 ulp of the result
    err = np.abs(got - Cs)
    assert np.all(err <= tol), f"{np.count_nonzero(err > tol)} outside tolerance, worst ratio {np.max(err / tol):.3g}"


@pytest.mark.parametrize("w_is_nk", [0, 1])
@pytest.mark.parametrize("Mn", [16, 64])
def test_config5_narrow_products_full_weight(Mn, w_is_nk):
    # the few-row products of the bench (decode phase of inference): Mn activation rows against the 8192 x 28672 weight, with
    # the workspace that makes the kernel deal equal ranges of the weight to all SMs (slabs cut between CTAs, four or two
    # MMA-issuing threads); sampled outputs, every row, against the FP64 oracle
    N, K = 28672, 8192
    g = _gen(987 + Mn)
    a = torch.randn(Mn, K, generator=g, device="cuda").to(torch.bfloat16)
    w = (torch.randn(K, N, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    Aq = torch.empty(Mn * K, dtype=torch.uint8, device="cuda")
    Wq = torch.empty(K * N, dtype=torch.uint8, device="cuda")
    se = torch.zeros(2, dtype=torch.int32, device="cuda")
    wsb = H.hif8_workspace_bytes(H.WS_AMAX_SCALE_ENCODE, 0)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    H.hif8_amax_scale_encode(a, H.BF16, Aq, Mn * K, 14, H.RND_TA, 0, 0, None, None, se[0:1], None, ws, wsb)
    H.hif8_amax_scale_encode(w, H.BF16, Wq, K * N, 14, H.RND_TA, 0, 0, None, None, se[1:2], None, ws, wsb)
    del a, w
    Wdev = Wq.view(K, N).t().contiguous().view(-1) if w_is_nk else Wq
    C = torch.full((Mn, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    gb = H.hif8_workspace_bytes(H.WS_GEMM, Mn * K + K * N)
    gws = torch.empty(gb, dtype=torch.uint8, device="cuda")
    H.hif8_gemm(Aq, K, Wdev, K if w_is_nk else N, w_is_nk, C, N, H.BF16, Mn, N, K, se[0:1], se[1:2], gws, gb)
    assert H.hif8_last_device_status() == 0
    sa, sw = [int(v) for v in se.cpu()]
    rng = np.random.default_rng(5)
    # random entries, the last slab, and the columns around a slab boundary that a range boundary cuts
    cols = np.concatenate([rng.integers(0, N, 40000), np.tile(np.arange(N - 128, N), Mn), np.tile(np.arange(96 * 128 - 64, 96 * 128 + 64), Mn)])
    rows = np.concatenate([rng.integers(0, Mn, 40000), np.repeat(np.arange(Mn), 128), np.repeat(np.arange(Mn), 128)])
    Cs, S = O.gemm_entries(Aq.cpu().numpy().reshape(Mn, K), Wq.cpu().numpy().reshape(K, N), False, sa, sw, rows, cols)
    got = C[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()].float().cpu().numpy().astype(np.float64)
    tol = 1e-5 * S
    tol = tol + 2.0 ** (np.floor(np.log2(np.maximum(np.abs(Cs) + tol, 2.0 ** -126))) - 8)   # + half a BF16 ulp of the result
    err = np.abs(got - Cs)
    assert np.all(err <= tol), f"{np.count_nonzero(err > tol)} outside tolerance, worst ratio {np.max(err / tol):.3g}"
    assert not torch.isnan(C.float()).any()                  # every output was written
