"""GPU parity of hif8_gemm (through the C ABI) against the FP64 oracle.

Tolerance (per output, from the method's statement): FP32 output |C - C*| <= 1e-5 * S with
S = 2^-(sa+sw) * sum_k |a_k w_k|; BF16 output additionally gets the one rounding to BF16 (round to nearest: half a
unit in the last place of the 8-bit significand, taken at the binade of the FP32 result, which lies within 1e-5 * S of C*).
"""
import numpy as np
import pytest
import torch

import paper_2409_16626_b200 as H
import workloads as W
from oracle import hif8_oracle as O

from gpu_util import bf16_half_ulp, to_dev

pytestmark = pytest.mark.gpu


def run_gemm(Aq, Wq, w_is_nk, c_dtype, sa=None, sw=None, M=None, N=None, K=None, lda=None, ldw=None, staged=False):
    M = Aq.shape[0] if M is None else M
    K = Aq.shape[1] if K is None else K
    N = (Wq.shape[0] if w_is_nk else Wq.shape[1]) if N is None else N
    dA, dW = to_dev(Aq), to_dev(Wq)
    ldc = (N + 7) // 8 * 8
    C = torch.full((M, ldc), float("nan"), dtype=torch.float32 if c_dtype == H.F32 else torch.bfloat16, device="cuda")
    # staged = True: workspace with room for both operands in BF16 -> decode-once path; "a": room for A alone -> A expanded
    # once, W decoded inside the tensor-core kernel; False: the fused kernel decodes both
    wsb = H.hif8_workspace_bytes(H.WS_GEMM, M * K if staged == "a" else M * K + K * N) if staged else H.hif8_workspace_bytes(H.WS_GEMM, 0)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    dsa = torch.tensor([sa], dtype=torch.int32, device="cuda") if sa is not None else None
    dsw = torch.tensor([sw], dtype=torch.int32, device="cuda") if sw is not None else None
    # (staged = True means the kernel that takes both operands expanded, whatever the size of the product)
    before = H.hif8_gemm_path_policy(H.GEMM_PATH_EXPAND_BOTH if staged is True else H.GEMM_PATH_AUTO)
    try:
        H.hif8_gemm(dA, Aq.shape[1] if lda is None else lda, dW, Wq.shape[1] if ldw is None else ldw, int(w_is_nk), C, ldc,
                    c_dtype, M, N, K, dsa, dsw, ws, wsb)
    finally:
        H.hif8_gemm_path_policy(before)
    assert H.hif8_gemm_status(ws) == 0
    out = C.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isnan(out[:, N:]))                      # padding columns untouched
    return out[:, :N]


def check(C, Cstar, S, c_dtype):
    tol = 1e-5 * S
    if c_dtype == H.BF16:
        tol = tol + bf16_half_ulp(np.abs(Cstar) + tol)
    err = np.abs(C - Cstar)
    bad = err > tol
    assert not bad.any(), f"{bad.sum()} of {bad.size} outside tolerance; worst ratio {np.max(err / np.maximum(tol, 1e-300)):.3g}"


@pytest.mark.parametrize("staged", [False, True, "a"])
@pytest.mark.parametrize("w_is_nk", [0, 1])
@pytest.mark.parametrize("c_dtype", [H.F32, H.BF16])
@pytest.mark.parametrize("shape", [(128, 256, 64), (128, 256, 256), (256, 512, 192), (130, 264, 208), (77, 40, 16),
                                   (300, 1000, 1040)])
def test_gemm_small_full_compare(shape, c_dtype, w_is_nk, staged):
    M, N, K = shape
    Aq = W.random_codes((M, K), seed=M + K)
    Wkn = W.random_codes((K, N), seed=N + K + 1)
    Wq = np.ascontiguousarray(Wkn.T) if w_is_nk else Wkn
    if (Wq.shape[1] % 16) != 0:                              # leading dimension must be a multiple of 16 bytes
        pad = 16 - Wq.shape[1] % 16
        Wq = np.ascontiguousarray(np.pad(Wq, ((0, 0), (0, pad))))
    Cs, S = O.gemm_full(Aq, Wkn, False, 0, 0)
    C = run_gemm(Aq, Wq, w_is_nk, c_dtype, N=N, staged=staged)
    check(C, Cs, S, c_dtype)


@pytest.mark.parametrize("staged", [False, True, "a"])
@pytest.mark.parametrize("w_is_nk", [0, 1])
def test_gemm_one_hot_rows_pin_tile_and_k_indexing(w_is_nk, staged):
    # A picks one k per row (value 1.0): C[m, :] must equal row perm[m] of W exactly
    M, N, K = 384, 768, 512
    rng = np.random.default_rng(5)
    perm = rng.integers(0, K, M)
    Aq = np.zeros((M, K), dtype=np.uint8)
    Aq[np.arange(M), perm] = 0x08
    Wkn = W.random_codes((K, N), seed=9)
    tab = np.array([O.value(c) for c in range(256)])
    C = run_gemm(Aq, np.ascontiguousarray(Wkn.T) if w_is_nk else Wkn, w_is_nk, H.F32, staged=staged)
    assert np.array_equal(C, tab[Wkn][perm, :])
    # and the mirror: W picks one k per column
    permn = rng.integers(0, K, N)
    Wsel = np.zeros((K, N), dtype=np.uint8)
    Wsel[permn, np.arange(N)] = 0x90                          # -2.0
    Aq2 = W.random_codes((M, K), seed=10)
    C = run_gemm(Aq2, np.ascontiguousarray(Wsel.T) if w_is_nk else Wsel, w_is_nk, H.F32, staged=staged)
    assert np.array_equal(C, -2.0 * tab[Aq2][:, permn])


def test_gemm_small_integers_exact_and_descale():
    M, N, K = 256, 256, 1024
    ints = np.array([0x00, 0x08, 0x10, 0x14, 0x20, 0x88, 0x90, 0x94], dtype=np.uint8)   # 0, 1, 2, 3, 4, -1, -2, -3
    rng = np.random.default_rng(3)
    Aq = ints[rng.integers(0, len(ints), (M, K))]
    Wq = ints[rng.integers(0, len(ints), (K, N))]
    tab = np.array([O.value(c) for c in range(256)])
    want = (tab[Aq].astype(np.int64) @ tab[Wq].astype(np.int64)).astype(np.float64)
    assert np.array_equal(run_gemm(Aq, Wq, 0, H.F32), want)
    assert np.array_equal(run_gemm(Aq, Wq, 0, H.F32, staged=True), want)
    assert np.array_equal(run_gemm(Aq, Wq, 0, H.F32, sa=-7, sw=2, staged=True), want * 32.0)
    assert np.array_equal(run_gemm(Aq, Wq, 0, H.F32, sa=3, sw=-1), want / 4.0)
    assert np.array_equal(run_gemm(Aq, Wq, 0, H.F32, sa=60, sw=55), want * 2.0 ** -115)


@pytest.mark.parametrize("M", [128, 16])
def test_gemm_specials_propagate(M):
    # (16 rows: the narrow kernel, whose activations are expanded by its preparing launch when the workspace has room)
    N, K = 256, 64
    Aq = np.full((M, K), 0x08, dtype=np.uint8)
    Wq = np.full((K, N), 0x08, dtype=np.uint8)
    Aq[3, 5] = 0x80                                           # NaN
    Aq[7, 9] = 0x6F                                           # +Inf
    for staged in (False, True, "a"):
        C = run_gemm(Aq, Wq, 0, H.F32, staged=staged)
        assert np.all(np.isnan(C[3])) and np.all(np.isposinf(C[7]))
        ok = np.ones(M, bool); ok[[3, 7]] = False
        assert np.all(C[ok] == K)


@pytest.mark.parametrize("w_is_nk", [0, 1])
def test_gemm_medium_scaled_operands_sampled(w_is_nk):
    # operands produced the way the method uses them: BF16 tensors, per-tensor scaled, encoded on the device
    M, N, K = 1024, 1536, 4096
    a = W.normal_bf16((M, K), seed=4567)
    w = W.normal_bf16((K, N), seed=5678, std=0.02)
    sa, sw = O.amax_scale(a, O.BF16, 14)[1], O.amax_scale(w, O.BF16, 14)[1]
    Aq = O.encode(a, O.BF16, sa, O.TA, 0, quick=True)
    Wkn = O.encode(w, O.BF16, sw, O.TA, 0, quick=True)
    rng = np.random.default_rng(1)
    rows = np.concatenate([rng.integers(0, M, 20000), np.repeat(np.arange(128), 256), np.repeat(np.arange(M - 128, M), 256)])
    cols = np.concatenate([rng.integers(0, N, 20000), np.tile(np.arange(256), 128), np.tile(np.arange(N - 256, N), 128)])
    Cs, S = O.gemm_entries(Aq, Wkn, False, sa, sw, rows, cols)
    for c_dtype in (H.F32, H.BF16):
        for staged in (False, True, "a"):
            C = run_gemm(Aq, np.ascontiguousarray(Wkn.T) if w_is_nk else Wkn, w_is_nk, c_dtype, sa=sa, sw=sw, staged=staged)
            check(C[rows, cols], Cs, S, c_dtype)


def _same_sign_operands(M, N, K, relu_only):
    """Codes of non-negative activations (|N(0,1)|, or max(N(0,1), 0) with `relu_only`) and of positive (or, with
    `relu_only`, zero-mean) N(0, 0.02) weights, per-tensor scaled to target exponent 14 and rounded half away."""
    a = W.bf16_bits_to_f32(W.normal_bf16((M, K), seed=4567))
    w = W.bf16_bits_to_f32(W.normal_bf16((K, N), seed=5678, std=0.02))
    a = np.maximum(a, 0.0) if relu_only else np.abs(a)
    if not relu_only:
        w = np.abs(w)
    ab, wb = W.f32_to_bf16_bits(a), W.f32_to_bf16_bits(w)
    sa, sw = O.amax_scale(ab, O.BF16, 14)[1], O.amax_scale(wb, O.BF16, 14)[1]
    return O.encode(ab, O.BF16, sa, O.TA, 0, quick=True), O.encode(wb, O.BF16, sw, O.TA, 0, quick=True), sa, sw


@pytest.mark.parametrize("relu_only", [False, True])
@pytest.mark.parametrize("path", ["fused", "staged", "a_expanded", "narrow"])
def test_gemm_same_sign_operands_k8192(path, relu_only):
    # Section 4.1: activations are GEMM inputs, and activations behind a ReLU are non-negative.  With operands of one
    # sign nothing cancels, S equals |C*|, and 512 sequential FP32 accumulator updates per output must stay inside
    # 1e-5 * S with no further allowance (FP32 output).
    M, N, K = (16 if path == "narrow" else 256), 512, 8192
    Aq, Wkn, sa, sw = _same_sign_operands(M, N, K, relu_only)
    Cs, S = O.gemm_full(Aq, Wkn, False, sa, sw)
    if not relu_only:
        assert np.allclose(Cs, S, rtol=1e-12)
    C = run_gemm(Aq, Wkn, 0, H.F32, sa=sa, sw=sw, staged={"staged": True, "a_expanded": "a"}.get(path, False))
    ratio = np.max(np.abs(C - Cs) / (1e-5 * S))
    print(f"same-sign K=8192 {path} relu_only={relu_only}: worst |err| / (1e-5 S) = {ratio:.3f}")
    assert ratio <= 1.0, ratio


def test_bounded_wait_gives_up_and_reports_without_disturbing_the_device():
    # failure detection: a wait that nothing satisfies runs out after its limit (50 ms here), the status word says so,
    # and the next GEMM on the same device works
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    H.hif8_selftest_wait_timeout(ws, 50)
    assert H.hif8_gemm_status(ws) == 10                      # HIF8_ERR_DEVICE_TIMEOUT
    assert H.hif8_last_device_status() == 10                 # the same word, found through the stream
    assert int(ws[:4].view(torch.int32).item()) == 99        # where it gave up
    M, N, K = 128, 256, 64
    Aq = np.full((M, K), 0x08, dtype=np.uint8)
    Wq = np.full((K, N), 0x10, dtype=np.uint8)
    assert np.all(run_gemm(Aq, Wq, 0, H.F32) == 2.0 * K)
    assert H.hif8_last_device_status() == 0                  # now the status word of that GEMM


@pytest.mark.parametrize("w_is_nk", [0, 1])
@pytest.mark.parametrize("c_dtype", [H.F32, H.BF16])
@pytest.mark.parametrize("staged", [False, True])
@pytest.mark.parametrize("shape", [(1, 256, 64), (16, 1008, 272), (17, 640, 1040), (33, 128, 16), (64, 400, 208), (48, 2064, 4096),
                                   (8, 304, 8192), (20, 912, 1472), (64, 1296, 2048), (16, 1168, 2432), (40, 1168, 2368)])
def test_gemm_narrow_products(shape, c_dtype, w_is_nk, staged):
    # M <= 64: the weight-streaming kernel (weights as the 128-row tensor-core operand, C accumulated transposed).
    # staged: with a workspace for partial sums the (slab, two-k-block unit) pairs are dealt out in equal contiguous ranges, so
    # slabs are cut (16, ~3 and 4 contributors per slab) and summed from per-contributor slices.  The last two shapes have 19
    # units per slab against ranges of 4.04 units: range and slab boundaries never line up, segments come as short as one
    # unit (fewer k-blocks than MMA-issuing threads: four, or two for more than 32 rows against [K,N] weights), and K = 2368 ends in half a unit.
    M, N, K = shape
    N16 = (N + 15) // 16 * 16
    Aq = W.random_codes((M, K), seed=M + K)
    Wkn = W.random_codes((K, N), seed=N + K + 3)
    for t in (Aq, Wkn):
        t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x33
    if w_is_nk:
        Wq = np.ascontiguousarray(Wkn.T)
    else:
        Wq = np.full((K, N16 + 16), 0x7B, dtype=np.uint8)     # padded leading dimension; the padding must not be read in
        Wq[:, :N] = Wkn
    Cs, S = O.gemm_full(Aq, Wkn, False, 3, -5)
    out = run_gemm(Aq, Wq, w_is_nk, c_dtype, sa=3, sw=-5, M=M, N=N, K=K, ldw=Wq.shape[1], staged=staged)
    check(out, Cs, S, c_dtype)
    if staged:  # slices are added in contributor order: the result does not depend on which CTA arrives last
        again = run_gemm(Aq, Wq, w_is_nk, c_dtype, sa=3, sw=-5, M=M, N=N, K=K, ldw=Wq.shape[1], staged=staged)
        assert np.array_equal(out, again)


@pytest.mark.parametrize("w_is_nk", [0, 1])
@pytest.mark.parametrize("form", ["padded_lda", "room_for_a_only"])
def test_gemm_narrow_activation_forms(form, w_is_nk):
    # With a workspace the narrow kernel takes its activations expanded to BF16 by a launch in front of it -- unless A has a
    # padded leading dimension (then the kernel decodes the activation bytes itself, with the slabs still cut between CTAs).
    # A workspace with room for A alone has no room for partial sums: expanded activations with one CTA per slab.
    M, N, K = 24, 1168, 2432
    Aq = W.random_codes((M, K), seed=5)
    Wkn = W.random_codes((K, N), seed=6)
    for t in (Aq, Wkn):
        t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x33
    Cs, S = O.gemm_full(Aq, Wkn, False, 1, 2)
    Wq = np.ascontiguousarray(Wkn.T) if w_is_nk else Wkn
    if form == "padded_lda":
        Ap = np.full((M, K + 32), 0x7B, dtype=np.uint8)
        Ap[:, :K] = Aq
        out = run_gemm(Ap, Wq, w_is_nk, H.F32, sa=1, sw=2, M=M, N=N, K=K, lda=K + 32, staged=True)
    else:
        out = run_gemm(Aq, Wq, w_is_nk, H.F32, sa=1, sw=2, M=M, N=N, K=K, staged="a")
    check(out, Cs, S, H.F32)


@pytest.mark.parametrize("K", [272, 2112])
def test_gemm_narrow_channel_scales_and_accumulate(K):
    # K = 2112 with the large workspace: slabs cut between CTAs, finished by whichever contributor arrives last
    M, N = 24, 528
    Aq = W.random_codes((M, K), seed=1)
    Wkn = W.random_codes((K, N), seed=2)
    for t in (Aq, Wkn):
        t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x33
    sw = np.random.default_rng(3).integers(-20, 20, size=N).astype(np.int32)
    c0 = (np.random.default_rng(4).standard_normal((M, N)) * 10).astype(np.float32)
    C = torch.from_numpy(c0.copy()).cuda()
    wsb = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N) if K > 1000 else 256
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    H.hif8_gemm_ex(to_dev(Aq), K, 0, to_dev(Wkn), N, 0, C, N, H.F32, M, N, K, torch.tensor([2], dtype=torch.int32, device="cuda"),
                   None, to_dev(sw.view(np.uint32)), 1, ws, wsb)
    assert H.hif8_gemm_status(ws) == 0
    rows, cols = np.divmod(np.arange(M * N), N)
    P, S = O.gemm_entries_channel(Aq, Wkn, 0, 2, sw, rows, cols)
    want = P.reshape(M, N) + c0
    assert np.all(np.abs(C.cpu().numpy().astype(np.float64) - want) <= 1e-5 * S.reshape(M, N) + 2.0 ** -24 * np.abs(want))


def test_gemm_calls_replay_from_a_cuda_graph():
    # the narrow call is two launches chained by programmatic stream serialization, the general one a memset node and a
    # cluster launch: both are captured into one graph and replayed on new operand contents
    M, N, K = 16, 1168, 2432
    M2 = 256
    dA, dW = torch.empty(M2 * K, dtype=torch.uint8, device="cuda"), torch.empty(K * N, dtype=torch.uint8, device="cuda")
    Cn = torch.zeros(M, N, dtype=torch.float32, device="cuda")
    Cg = torch.zeros(M2, N, dtype=torch.float32, device="cuda")
    wsb = H.hif8_workspace_bytes(H.WS_GEMM, M2 * K + K * N)
    ws_n, ws_g = torch.empty(wsb, dtype=torch.uint8, device="cuda"), torch.empty(wsb, dtype=torch.uint8, device="cuda")

    def calls():
        H.hif8_gemm(dA, K, dW, N, 0, Cn, N, H.F32, M, N, K, None, None, ws_n, wsb)
        H.hif8_gemm(dA, K, dW, N, 0, Cg, N, H.F32, M2, N, K, None, None, ws_g, 256)

    def load(seed):
        Aq, Wq = W.random_codes((M2, K), seed=seed), W.random_codes((K, N), seed=seed + 1)
        for t in (Aq, Wq):
            t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x33
        dA.copy_(torch.from_numpy(Aq.reshape(-1)))
        dW.copy_(torch.from_numpy(Wq.reshape(-1)))
        return Aq, Wq

    load(1)
    calls()                                                   # eager first: one-time set-up happens outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        calls()
    for seed in (7, 9):
        Aq, Wq = load(seed)
        g.replay()
        torch.cuda.synchronize()
        assert H.hif8_gemm_status(ws_n) == 0 and H.hif8_gemm_status(ws_g) == 0
        Cs, S = O.gemm_full(Aq, Wq, False, 0, 0)
        check(Cg.cpu().numpy().astype(np.float64), Cs, S, H.F32)
        check(Cn.cpu().numpy().astype(np.float64), Cs[:M], S[:M], H.F32)


def test_tensor_map_cache_survives_eviction_and_pointer_reuse():
    # more distinct (pointer, shape) pairs than the library's tensor-map cache holds, each product exact in small integers;
    # then the same device buffers again with other shapes and contents (a cached map must never serve a different tensor)
    ints = np.array([0x00, 0x08, 0x10, 0x14, 0x88, 0x90], dtype=np.uint8)          # 0, 1, 2, 3, -1, -2
    tab = np.array([O.value(c) for c in range(256)])
    rng = np.random.default_rng(11)
    bufA = torch.empty(512 * 1024, dtype=torch.uint8, device="cuda")
    bufW = torch.empty(1024 * 512, dtype=torch.uint8, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    stream2 = torch.cuda.Stream()
    for it in range(80):
        M, N, K = 16 * int(rng.integers(1, 20)), 16 * int(rng.integers(1, 24)), 16 * int(rng.integers(1, 40))
        Aq = ints[rng.integers(0, len(ints), (M, K))]
        Wq = ints[rng.integers(0, len(ints), (K, N))]
        bufA[:M * K].copy_(torch.from_numpy(Aq.reshape(-1)))
        bufW[:K * N].copy_(torch.from_numpy(Wq.reshape(-1)))
        C = torch.zeros(M, N, dtype=torch.float32, device="cuda")
        st = stream2 if it % 3 == 0 else None
        if st is not None:
            st.wait_stream(torch.cuda.current_stream())
        H.hif8_gemm(bufA, K, bufW, N, 0, C, N, H.F32, M, N, K, None, None, ws, 256, stream=st)
        assert H.hif8_last_device_status(st) == 0            # synchronises that stream
        want = (tab[Aq].astype(np.int64) @ tab[Wq].astype(np.int64)).astype(np.float64)
        assert np.array_equal(C.cpu().numpy().astype(np.float64), want), (it, M, N, K)
    assert H.hif8_last_device_status(torch.cuda.Stream()) == 0   # a stream that never saw a GEMM


@pytest.mark.parametrize("mode", ["fused", "a", "a_nk", "staged"])
def test_gemm_repeated_runs_are_bit_identical(mode):
    # The order of the sums is fixed (k-blocks in order, one accumulator per output), so repeated runs of one product must
    # agree bit for bit; an operand tile handed to the tensor core before its last byte was in place -- the hand-over between
    # the decode warps of both CTAs of a pair and the MMA thread -- would show as a difference in some run.  Full tiles, many
    # k-blocks, every general kernel; the first run is checked against the oracle on sampled outputs.
    M, N, K = 1024, 2048, 8192
    Aq = W.random_codes((M, K), seed=77)
    Wkn = W.random_codes((K, N), seed=78)
    for t in (Aq, Wkn):
        t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x21
    w_is_nk = mode == "a_nk"
    Wq = np.ascontiguousarray(Wkn.T) if w_is_nk else Wkn
    staged = {"fused": False, "a": "a", "a_nk": "a", "staged": True}[mode]
    first = run_gemm(Aq, Wq, w_is_nk, H.F32, sa=2, sw=-3, staged=staged)
    rng = np.random.default_rng(9)
    rows, cols = rng.integers(0, M, 4000), rng.integers(0, N, 4000)
    Cs, S = O.gemm_entries(Aq, Wkn, False, 2, -3, rows, cols)
    assert np.all(np.abs(first[rows, cols] - Cs) <= 1e-5 * S)
    for _ in range(8):
        again = run_gemm(Aq, Wq, w_is_nk, H.F32, sa=2, sw=-3, staged=staged)
        assert np.array_equal(first, again)
