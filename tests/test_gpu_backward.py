"""GPU parity (through the C ABI) of the backward-pass operand forms: conversion with transposed store, and the general
GEMM entry (A read as [K,M], weights as [N,K], accumulation into C) against the oracle.  Section 3 (TA or hybrid rounding
in the backward pass), Section 4.1 (activation gradients are GEMM inputs), Algorithm 1 ("MatMul & Restore")."""
import numpy as np
import pytest
import torch

import paper_2409_16626_b200 as H
import workloads as W
from oracle import hif8_oracle as O

from gpu_util import bf16_half_ulp, both_operands_expanded, dev_empty, to_dev

pytestmark = pytest.mark.gpu


def source(rows, cols, seed, dtype):
    x = W.loguniform_f32(rows * cols, seed).reshape(rows, cols)
    if rows > 4 and cols > 4:
        x[1, 2] = np.inf
        x[2, 3] = np.nan
        x[3, 1] = -0.0
    if dtype == H.F32:
        return x
    if dtype == H.BF16:
        return W.f32_to_bf16_bits(x)
    with np.errstate(over="ignore"):
        return x.astype(np.float16).view(np.uint16)


def run_transpose(x, dtype, scale_exp=0, rnd=H.RND_TA, flags=0, seed=0, dev_exp=None, offset=0):
    rows, cols = x.shape
    raw = np.ascontiguousarray(x).view(np.uint8).ravel()
    buf = torch.zeros(raw.size + offset + 16, dtype=torch.uint8, device="cuda")
    buf[offset:offset + raw.size] = torch.from_numpy(raw.copy()).cuda()
    owner, dptr, read = dev_empty(rows * cols, np.uint8)
    d_exp = torch.tensor([dev_exp], dtype=torch.int32, device="cuda") if dev_exp is not None else None
    H.hif8_encode_transpose(buf.data_ptr() + offset, dtype, dptr, rows, cols, scale_exp, d_exp, rnd, flags, seed)
    torch.cuda.synchronize()
    return read().reshape(cols, rows)


@pytest.mark.parametrize("dtype", [H.F32, H.BF16, H.F16])
@pytest.mark.parametrize("shape", [(256, 128), (144, 72), (1040, 520), (16, 8), (130, 50), (48, 4096), (2064, 7048), (4112, 14360)])
def test_encode_transpose_matches_oracle(shape, dtype):
    # the last two shapes are large enough for two and for four column strips per block (ragged in both directions)
    x = source(*shape, seed=shape[0], dtype=dtype)
    se = 30 if dtype != H.F16 else 3
    q = run_transpose(x, dtype, scale_exp=se, rnd=H.RND_HR)
    assert np.array_equal(q, O.encode_transpose(x, dtype, se, O.HR, quick=True))


@pytest.mark.parametrize("mode", [H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR])
@pytest.mark.parametrize("dtype", [H.F32, H.BF16])
def test_encode_transpose_modes_flags_device_exponent_and_misalignment(dtype, mode):
    x = source(272, 136, seed=7, dtype=dtype)
    flags = H.FLAG_SATURATE | H.FLAG_NAN_TO_ZERO
    q = run_transpose(x, dtype, scale_exp=99, rnd=mode, flags=flags, seed=31, dev_exp=25)  # the device exponent wins
    ref = O.encode_transpose(x, dtype, 25, mode, flags, 31, quick=True)
    assert np.array_equal(q, ref)
    q2 = run_transpose(x, dtype, scale_exp=25, rnd=mode, flags=flags, seed=31, offset=4 if dtype == H.F32 else 2)
    assert np.array_equal(q2, ref)
    # the same codes as the flat encoder, moved
    flat = torch.empty(x.size, dtype=torch.uint8, device="cuda")
    H.hif8_encode(to_dev(x), dtype, flat, x.size, 25, mode, flags, 31)
    assert np.array_equal(flat.cpu().numpy().reshape(x.shape).T, q)


@pytest.mark.parametrize("flags", [0, H.FLAG_SATURATE | H.FLAG_NAN_TO_ZERO])
@pytest.mark.parametrize("dtype", [H.BF16, H.F16])
def test_encode_transpose_every_16_bit_pattern(dtype, flags):
    # every sign, zero, subnormal, Inf and NaN pattern through the tiled kernel (Section 3: special values and options)
    x = np.arange(65536, dtype=np.uint16).reshape(256, 256)
    for mode, omode in ((H.RND_TA, O.TA), (H.RND_HR, O.HR), (H.RND_TE, O.TE)):
        for se in (0, -9):
            q = run_transpose(x, dtype, scale_exp=se, rnd=mode, flags=flags)
            assert np.array_equal(q, O.encode_transpose(x, dtype, se, omode, flags, 0, quick=True)), (mode, se)


def test_encode_transpose_argument_checks():
    x = torch.ones(64, device="cuda")
    out = torch.empty(64, dtype=torch.uint8, device="cuda")
    assert H.hif8_encode_transpose(x, H.F32, out, 0, 8) == 0
    assert H.hif8_encode_transpose(x, H.F32, out, -1, 8, check=False) == 6
    assert H.hif8_encode_transpose(x, H.F32, out, 8, 8, scale_exp=127, check=False) == 5
    assert H.hif8_encode_transpose(None, H.F32, out, 8, 8, check=False) == 1
    assert H.hif8_encode_transpose(x, 5, out, 8, 8, check=False) == 2
    assert H.hif8_encode_transpose(x, H.F32, out, 8, 8, rnd=9, check=False) == 3


def codes(shape, seed):
    q = W.random_codes(shape, seed=seed)
    q[(q == 0x80) | ((q & 0x7F) == 0x6F)] = 0x15
    return q


@pytest.mark.parametrize("staged", [False, True, "a"])  # "a": workspace for A alone (A expanded once, W decoded in the kernel)
@pytest.mark.parametrize("a_is_km,w_is_nk", [(1, 0), (1, 1), (0, 1)])
@pytest.mark.parametrize("c_dtype,accumulate", [(H.F32, 0), (H.F32, 1), (H.BF16, 1)])
def test_gemm_ex_layouts_and_accumulate(c_dtype, accumulate, a_is_km, w_is_nk, staged):
    M, N, K = 208, 528, 272
    Amk, Wkn = codes((M, K), 5), codes((K, N), 6)
    Aq = np.ascontiguousarray(Amk.T) if a_is_km else Amk
    Wq = np.ascontiguousarray(Wkn.T) if w_is_nk else Wkn
    sa, sw = 4, -9
    ldc = N + 8
    rng = np.random.default_rng(3)
    c0 = (rng.standard_normal((M, ldc)) * 50).astype(np.float32)
    C = torch.from_numpy(c0).cuda().to(torch.float32 if c_dtype == H.F32 else torch.bfloat16)
    c0 = C.float().cpu().numpy().astype(np.float64)
    wsb = H.hif8_workspace_bytes(H.WS_GEMM, (M * K if staged == "a" else M * K + K * N) if staged else 0)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    with both_operands_expanded(staged is True):
        H.hif8_gemm_ex(to_dev(Aq), Aq.shape[1], a_is_km, to_dev(Wq), Wq.shape[1], w_is_nk, C, ldc, c_dtype, M, N, K,
                       torch.tensor([sa], dtype=torch.int32, device="cuda"), torch.tensor([sw], dtype=torch.int32, device="cuda"),
                       None, accumulate, ws, wsb)
    assert H.hif8_gemm_status(ws) == 0
    out = C.float().cpu().numpy().astype(np.float64)
    assert np.array_equal(out[:, N:], c0[:, N:])             # padding columns untouched
    rows, cols = np.divmod(np.arange(M * N), N)
    P, S = O.gemm_entries_ex(Aq, a_is_km, Wq, w_is_nk, sa, sw, rows, cols)
    P, S = P.reshape(M, N), S.reshape(M, N)
    Cs = P + (c0[:, :N] if accumulate else 0.0)
    # product within 1e-5 S; the accumulation adds one FP32 rounding of the sum; BF16 output its final rounding
    tol = 1e-5 * S + (2.0 ** -24 * np.abs(Cs) if accumulate else 0.0)
    if c_dtype == H.BF16:
        tol = tol + bf16_half_ulp(np.abs(Cs) + tol)
    assert np.all(np.abs(out[:, :N] - Cs) <= tol)


def test_gemm_ex_channel_exponents_with_transposed_a():
    M, N, K = 128, 256, 64
    Amk, Wkn = codes((M, K), 8), codes((K, N), 9)
    sw = np.random.default_rng(5).integers(-12, 12, size=N).astype(np.int32)
    C = torch.zeros(M, N, dtype=torch.float32, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    H.hif8_gemm_ex(to_dev(np.ascontiguousarray(Amk.T)), M, 1, to_dev(Wkn), N, 0, C, N, H.F32, M, N, K, None,
                   torch.tensor([99], dtype=torch.int32, device="cuda"), to_dev(sw.view(np.uint32)), 0, ws, 256)
    assert H.hif8_gemm_status(ws) == 0
    rows, cols = np.divmod(np.arange(M * N), N)
    P, S = O.gemm_entries_ex(np.ascontiguousarray(Amk.T), 1, Wkn, 0, 0, sw, rows, cols)  # the channel array wins over d_sw
    assert np.all(np.abs(C.cpu().numpy().astype(np.float64).ravel() - P) <= 1e-5 * S)


def test_backward_pass_of_a_linear_layer():
    # Y = X W; dX = dY W^T (dgrad), dW = X^T dY (wgrad, accumulated over two micro-batches), all operands as HiF8
    # bytes produced once, no transposed copies: X [Mb,K], W [K,N], dY [Mb,N]
    Mb, K, N = 256, 192, 320
    rng = np.random.default_rng(0)
    Wf = (rng.standard_normal((K, N)) * 0.05).astype(np.float32)
    qW, sW = None, None
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    dqW = torch.empty(K * N, dtype=torch.uint8, device="cuda")
    dsW = torch.zeros(1, dtype=torch.int32, device="cuda")
    H.hif8_amax_scale_encode(to_dev(Wf), H.F32, dqW, K * N, 2, H.RND_TA, 0, 0, None, None, dsW, None, ws, 256)
    sW = O.amax_scale(Wf, O.F32, 2)[1]
    qW = O.encode(Wf.ravel(), O.F32, sW, O.TA).reshape(K, N)
    assert np.array_equal(dqW.cpu().numpy().reshape(K, N), qW)
    dW = torch.zeros(K, N, dtype=torch.float32, device="cuda")
    dW_ref = np.zeros((K, N))
    S_acc = np.zeros((K, N))
    gws = torch.empty(256, dtype=torch.uint8, device="cuda")
    for mb in range(2):
        X = (rng.standard_normal((Mb, K))).astype(np.float32)
        dY = (rng.standard_normal((Mb, N)) * 1e-3).astype(np.float32)
        dqX = torch.empty(Mb * K, dtype=torch.uint8, device="cuda")
        dqG = torch.empty(Mb * N, dtype=torch.uint8, device="cuda")
        dsX = torch.zeros(1, dtype=torch.int32, device="cuda")
        dsG = torch.zeros(1, dtype=torch.int32, device="cuda")
        H.hif8_amax_scale_encode(to_dev(X), H.F32, dqX, Mb * K, 2, H.RND_TA, 0, 0, None, None, dsX, None, ws, 256)
        H.hif8_amax_scale_encode(to_dev(dY), H.F32, dqG, Mb * N, 2, H.RND_HR, 0, 0, None, None, dsG, None, ws, 256)
        sX, sG = O.amax_scale(X, O.F32, 2)[1], O.amax_scale(dY, O.F32, 2)[1]
        qX = O.encode(X.ravel(), O.F32, sX, O.TA).reshape(Mb, K)
        qG = O.encode(dY.ravel(), O.F32, sG, O.HR).reshape(Mb, N)
        assert np.array_equal(dqX.cpu().numpy().reshape(Mb, K), qX) and np.array_equal(dqG.cpu().numpy().reshape(Mb, N), qG)
        # dgrad: [Mb,N] x [K,N]^T -> [Mb,K]; the forward weight bytes are the [N_out=K, K_c=N] operand
        dX = torch.empty(Mb, K, dtype=torch.float32, device="cuda")
        H.hif8_gemm_ex(dqG, N, 0, dqW, N, 1, dX, K, H.F32, Mb, K, N, dsG, dsW, None, 0, gws, 256)
        assert H.hif8_gemm_status(gws) == 0
        rows, cols = np.divmod(np.arange(Mb * K), K)
        P, S = O.gemm_entries_ex(qG, 0, qW, 1, sG, sW, rows, cols)
        assert np.all(np.abs(dX.cpu().numpy().astype(np.float64).ravel() - P) <= 1e-5 * S)
        exact = dY.astype(np.float64) @ Wf.astype(np.float64).T
        assert np.linalg.norm(P.reshape(Mb, K) - exact) / np.linalg.norm(exact) < 0.08
        # wgrad: X^T [K,Mb] x dY [Mb,N] -> [K,N], accumulated
        H.hif8_gemm_ex(dqX, K, 1, dqG, N, 0, dW, N, H.F32, K, N, Mb, dsX, dsG, None, 1, gws, 256)
        assert H.hif8_gemm_status(gws) == 0
        rows, cols = np.divmod(np.arange(K * N), N)
        P, S = O.gemm_entries_ex(qX, 1, qG, 0, sX, sG, rows, cols)
        dW_ref += P.reshape(K, N)
        S_acc += S.reshape(K, N)
    got = dW.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - dW_ref) <= 1e-5 * S_acc + 2.0 ** -23 * np.abs(dW_ref))


@pytest.mark.parametrize("shape", [(200, 72, 16), (56, 264, 80), (129, 8, 1040)])
@pytest.mark.parametrize("w_is_nk", [0, 1])
def test_gemm_ex_transposed_a_ragged_shapes_and_padded_leading_dimensions(shape, w_is_nk):
    # A stored [K, M] with lda > M, M not a multiple of anything convenient, tiny K / N: the fused kernel (operands not
    # contiguous), out-of-range parts of the TMA boxes must read as zero
    M, N, K = shape
    lda = (M + 15) // 16 * 16 + 16
    ldw = ((K if w_is_nk else N) + 15) // 16 * 16 + 16
    Amk, Wkn = codes((M, K), 21), codes((K, N), 22)
    Aq = np.full((K, lda), 0x7B, dtype=np.uint8)            # padding holds a large finite value: it must never be read in
    Aq[:, :M] = Amk.T
    Wsrc = Wkn.T if w_is_nk else Wkn
    Wq = np.full((Wsrc.shape[0], ldw), 0x7B, dtype=np.uint8)
    Wq[:, :Wsrc.shape[1]] = Wsrc
    ldc = (N + 7) // 8 * 8
    C = torch.full((M, ldc), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    H.hif8_gemm_ex(to_dev(Aq), lda, 1, to_dev(Wq), ldw, w_is_nk, C, ldc, H.F32, M, N, K, None, None, None, 0, ws, 256)
    assert H.hif8_gemm_status(ws) == 0
    out = C.cpu().numpy().astype(np.float64)
    assert np.all(np.isnan(out[:, N:]))
    rows, cols = np.divmod(np.arange(M * N), N)
    P, S = O.gemm_entries_ex(np.ascontiguousarray(Amk.T), 1, np.ascontiguousarray(Wsrc), w_is_nk, 0, 0, rows, cols)
    assert np.all(np.abs(out[:, :N].ravel() - P) <= 1e-5 * S)


def test_gemm_ex_argument_checks():
    A = torch.zeros(64 * 64, dtype=torch.uint8, device="cuda")
    C = torch.zeros(64 * 64, dtype=torch.float32, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    ok = dict(workspace=ws, workspace_bytes=256, check=False)
    assert H.hif8_gemm_ex(A, 64, 1, A, 64, 0, C, 64, H.F32, 64, 64, 64, **ok) == 0
    assert H.hif8_gemm_ex(A, 48, 1, A, 64, 0, C, 64, H.F32, 64, 64, 64, **ok) == 6    # lda < M for a [K,M] operand
    assert H.hif8_gemm_ex(A, 64, 1, A, 64, 0, C, 64, H.F32, 64, 64, 24, **ok) == 6    # K not a multiple of 16
    assert H.hif8_gemm_ex(A, 72, 1, A, 64, 0, C, 64, H.F32, 64, 64, 64, **ok) == 7    # lda not a multiple of 16
    assert H.hif8_gemm_ex(A, 64, 1, A, 64, 0, C, 64, 5, 64, 64, 64, **ok) == 2
    assert H.hif8_gemm_ex(A, 64, 1, A, 64, 0, C, 64, H.F32, 64, 64, 64, workspace=None, workspace_bytes=0, check=False) == 8
    assert H.hif8_gemm_ex(A, 64, 1, A, 64, 0, C, 64, H.F32, 0, 64, 64, **ok) == 0     # empty output
