"""GPU parity (through the C ABI) of per-channel weight scaling, the channel-scaled GEMM restore and the
every-N-iterations amax cadence (Section 5.1) against the oracle.  Conversions and exponents are bit-exact; the GEMM
uses the tolerance of the per-tensor GEMM tests."""
import numpy as np
import pytest
import torch

import paper_2409_16626_b200 as H
import workloads as W
from oracle import hif8_oracle as O

from gpu_util import NP_OF, bf16_half_ulp, both_operands_expanded, dev_empty, to_dev

pytestmark = pytest.mark.gpu
MODES = [H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR]


def weight(rows, cols, seed, dtype, specials=True):
    x = W.normal_f32(rows * cols, seed).reshape(rows, cols)
    rng = np.random.default_rng(seed)
    x *= np.exp2(rng.integers(-20, 20, size=(1, cols))).astype(np.float32)
    x *= np.exp2(rng.integers(-6, 6, size=(rows, 1))).astype(np.float32)
    if specials and rows > 8 and cols > 8:
        x[3, 5] = np.inf
        x[4, 7] = np.nan
        x[:, 2] = 0.0
        x[6, :] = 0.0
    if dtype == H.F32:
        return x
    if dtype == H.BF16:
        return W.f32_to_bf16_bits(x)
    with np.errstate(over="ignore"):
        return np.clip(x, -60000, 60000).astype(np.float16).view(np.uint16)


def run_channel(x, dtype, axis, rnd=H.RND_TA, flags=0, seed=0, target=14, given=None, offset=0):
    rows, cols = x.shape
    ch = rows if axis == 0 else cols
    item = 4 if dtype == H.F32 else 2
    raw = np.ascontiguousarray(x).view(np.uint8).ravel()
    buf = torch.zeros(raw.size + offset + 16, dtype=torch.uint8, device="cuda")
    buf[offset:offset + raw.size] = torch.from_numpy(raw.copy()).cuda()
    owner, dptr, read = dev_empty(rows * cols, np.uint8, offset_bytes=offset)
    d_amax = torch.full((ch,), -1.0, dtype=torch.float32, device="cuda")
    d_se = torch.full((ch,), 77, dtype=torch.int32, device="cuda")
    d_in = to_dev(np.asarray(given, dtype=np.int32).view(np.uint32)) if given is not None else None
    H.hif8_channel_amax_scale_encode(buf.data_ptr() + offset, dtype, dptr, rows, cols, axis, target, rnd, flags, seed, d_in,
                                     d_amax, d_se)
    torch.cuda.synchronize()
    assert item * rows * cols == raw.size
    return read().reshape(rows, cols), d_amax.cpu().numpy(), d_se.cpu().numpy()


@pytest.mark.parametrize("dtype", [H.F32, H.BF16, H.F16])
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", [(300, 520), (64, 4096), (1031, 264), (9, 8), (257, 40), (12, 20480)])
def test_channel_encode_ta_matches_oracle(shape, axis, dtype):
    x = weight(*shape, seed=shape[0] + axis, dtype=dtype)
    q, amax, se = run_channel(x, dtype, axis)
    amax_o, se_o = O.channel_amax_scale(x, dtype, axis, 14)
    assert np.array_equal(amax, amax_o) and np.array_equal(se, se_o)
    assert np.array_equal(q, O.channel_encode(x, dtype, axis, se_o, quick=True))


@pytest.mark.parametrize("dtype,shape", [(H.F32, (2400, 8192)), (H.BF16, (4096, 7168)), (H.BF16, (1216, 16384))])
@pytest.mark.parametrize("axis", [0, 1])
def test_channel_encode_large(axis, dtype, shape):
    # large enough for the widest column strips (8 and 4 warps across) and for rows of exactly one register tile
    x = weight(*shape, seed=21, dtype=dtype)
    q, amax, se = run_channel(x, dtype, axis, rnd=H.RND_HR)
    amax_o, se_o = O.channel_amax_scale(x, dtype, axis, 14)
    assert np.array_equal(amax, amax_o) and np.array_equal(se, se_o)
    assert np.array_equal(q, O.channel_encode(x, dtype, axis, se_o, rnd=H.RND_HR, quick=True))


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("dtype", [H.F32, H.BF16])
def test_channel_encode_all_modes_and_flags(dtype, axis, mode):
    x = weight(200, 328, seed=17, dtype=dtype)
    flags = H.FLAG_SATURATE | H.FLAG_NAN_TO_ZERO if mode in (H.RND_TA, H.RND_SR) else 0
    q, _, se = run_channel(x, dtype, axis, rnd=mode, flags=flags, seed=99, target=9)
    _, se_o = O.channel_amax_scale(x, dtype, axis, 9)
    assert np.array_equal(se, se_o)
    assert np.array_equal(q, O.channel_encode(x, dtype, axis, se_o, rnd=mode, flags=flags, seed=99, quick=True))


@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("dtype", [H.F32, H.BF16])
def test_channel_encode_given_exponents_and_odd_layouts(dtype, axis):
    # cols not a multiple of the vector width, and a misaligned base pointer: the element-wise path, same results
    for shape, offset in (((70, 131), 0), ((40, 256), 4 if dtype == H.F32 else 2)):
        x = weight(*shape, seed=5, dtype=dtype)
        ch = shape[axis]
        given = np.random.default_rng(1).integers(-30, 30, size=ch).astype(np.int32)
        q, amax, se = run_channel(x, dtype, axis, rnd=H.RND_HR, given=given, offset=offset)
        assert np.array_equal(se, given) and np.all(amax == -1.0)  # amax untouched when the exponents are given
        assert np.array_equal(q, O.channel_encode(x, dtype, axis, given, rnd=H.RND_HR, quick=True))
        q2, amax2, se2 = run_channel(x, dtype, axis, offset=offset)
        amax_o, se_o = O.channel_amax_scale(x, dtype, axis, 14)
        assert np.array_equal(amax2, amax_o) and np.array_equal(se2, se_o)
        assert np.array_equal(q2, O.channel_encode(x, dtype, axis, se_o, quick=True))


def test_channel_encode_degenerate_shapes():
    d_amax = torch.full((5,), -1.0, device="cuda")
    d_se = torch.full((5,), 9, dtype=torch.int32, device="cuda")
    assert H.hif8_channel_amax_scale_encode(None, H.F32, None, 5, 0, 0, d_amax=d_amax, d_scale_exp_out=d_se) == 0
    torch.cuda.synchronize()
    assert d_amax.cpu().tolist() == [0.0] * 5 and d_se.cpu().tolist() == [0] * 5
    assert H.hif8_channel_amax_scale_encode(None, H.F32, None, 0, 7, 0) == 0
    x = to_dev(np.ones((4, 4), dtype=np.float32))
    out = torch.empty(16, dtype=torch.uint8, device="cuda")
    assert H.hif8_channel_amax_scale_encode(x, H.F32, out, 4, 4, 2, d_amax=d_amax, check=False) == 6   # axis
    assert H.hif8_channel_amax_scale_encode(x, H.F32, out, 4, 4, 1, check=False) == 1                   # no amax array
    assert H.hif8_channel_amax_scale_encode(x, 7, out, 4, 4, 1, d_amax=d_amax, check=False) == 2


@pytest.mark.parametrize("staged", [False, True, "a"])  # "a": workspace for A alone (with [N,K] weights: the swapped form,
                                                        # one weight exponent per accumulator row)
@pytest.mark.parametrize("w_is_nk", [0, 1])
@pytest.mark.parametrize("c_dtype", [H.F32, H.BF16])
def test_gemm_channel_scaled(c_dtype, w_is_nk, staged):
    M, N, K = 200, 528, 272
    Aq = W.random_codes((M, K), seed=3)
    Wkn = W.random_codes((K, N), seed=4)
    for t in (Aq, Wkn):
        t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x12
    Wq = np.ascontiguousarray(Wkn.T) if w_is_nk else Wkn
    sw = np.random.default_rng(8).integers(-25, 25, size=N).astype(np.int32)
    sa = -7
    ldc = (N + 7) // 8 * 8
    C = torch.full((M, ldc), float("nan"), dtype=torch.float32 if c_dtype == H.F32 else torch.bfloat16, device="cuda")
    wsb = H.hif8_workspace_bytes(H.WS_GEMM, (M * K if staged == "a" else M * K + K * N) if staged else 0)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    with both_operands_expanded(staged is True):
        H.hif8_gemm_channel_scaled(to_dev(Aq), K, to_dev(Wq), Wq.shape[1], w_is_nk, C, ldc, c_dtype, M, N, K,
                                   torch.tensor([sa], dtype=torch.int32, device="cuda"), to_dev(sw.view(np.uint32)), ws, wsb)
    assert H.hif8_gemm_status(ws) == 0
    out = C.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isnan(out[:, N:]))
    rows, cols = np.divmod(np.arange(M * N), N)
    Cs, S = O.gemm_entries_channel(Aq, Wq, w_is_nk, sa, sw, rows, cols)
    Cs, S = Cs.reshape(M, N), S.reshape(M, N)
    tol = 1e-5 * S
    if c_dtype == H.BF16:
        tol = tol + bf16_half_ulp(np.abs(Cs) + tol)
    assert np.all(np.abs(out[:, :N] - Cs) <= tol)


def test_channel_pipeline_weight_to_gemm():
    # (target exponent 2: amax lands in [4, 8), where HiF8 is most precise)
    # the whole use: per-channel encode of a [K,N] weight, per-tensor encode of the activation, channel-scaled GEMM;
    # the result approximates the unquantized product and equals the oracle's pipeline within the GEMM tolerance
    M, N, K = 96, 256, 512
    a = W.normal_f32(M * K, 1).reshape(M, K)
    w = weight(K, N, seed=2, dtype=H.F32, specials=False)
    qa_o = O.encode(a.ravel(), O.F32, O.amax_scale(a.ravel(), O.F32, 2)[1]).reshape(M, K)
    sa_o = O.amax_scale(a.ravel(), O.F32, 2)[1]
    _, sw_o = O.channel_amax_scale(w, O.F32, 1, 2)
    qw_o = O.channel_encode(w, O.F32, 1, sw_o)
    dqa = torch.empty(M * K, dtype=torch.uint8, device="cuda")
    dqw = torch.empty(K * N, dtype=torch.uint8, device="cuda")
    dsa = torch.zeros(1, dtype=torch.int32, device="cuda")
    dsw = torch.zeros(N, dtype=torch.int32, device="cuda")
    damax = torch.zeros(N, dtype=torch.float32, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    H.hif8_amax_scale_encode(to_dev(a), H.F32, dqa, M * K, 2, H.RND_TA, 0, 0, None, None, dsa, None, ws, 256)
    H.hif8_channel_amax_scale_encode(to_dev(w), H.F32, dqw, K, N, 1, 2, H.RND_TA, 0, 0, None, damax, dsw)
    assert np.array_equal(dqa.cpu().numpy().reshape(M, K), qa_o) and np.array_equal(dqw.cpu().numpy().reshape(K, N), qw_o)
    C = torch.empty(M, N, dtype=torch.float32, device="cuda")
    gws = torch.empty(256, dtype=torch.uint8, device="cuda")
    H.hif8_gemm_channel_scaled(dqa, K, dqw, N, 0, C, N, H.F32, M, N, K, dsa, dsw, gws, 256)
    assert H.hif8_gemm_status(gws) == 0
    rows, cols = np.divmod(np.arange(M * N), N)
    Cs, S = O.gemm_entries_channel(qa_o, qw_o, 0, sa_o, sw_o, rows, cols)
    out = C.cpu().numpy().astype(np.float64).ravel()
    assert np.all(np.abs(out - Cs) <= 1e-5 * S)
    exact = a.astype(np.float64) @ w.astype(np.float64)
    rel = np.linalg.norm(out.reshape(M, N) - exact) / np.linalg.norm(exact)
    assert rel < 0.06  # target exponent 2 puts each channel's bulk into the 3-bit-mantissa binades (|E| <= 3)


@pytest.mark.parametrize("dtype,rnd", [(H.F32, H.RND_TA), (H.BF16, H.RND_HR), (H.F32, H.RND_HR), (H.BF16, H.RND_SSR)])
@pytest.mark.parametrize("interval,hist", [(1, 1), (3, 2), (10, 4)])
def test_delayed_scale_cadence(interval, hist, dtype, rnd):
    T, n = 24, 70001
    rng = np.random.default_rng(interval * 10 + hist)
    tensors = []
    for t in range(T):
        x = W.normal_f32(n, 500 + t) * np.float32(2.0 ** rng.integers(-12, 12))
        if t == 4:
            x[:] = 0.0                      # an all-zero tensor measures amax 0
        if t == 9:
            x[5] = np.inf                   # non-finite elements do not count
        tensors.append(x if dtype == H.F32 else W.f32_to_bf16_bits(x))
    amax = np.array([O.amax_scale(x, dtype, 14)[0] for x in tensors], dtype=np.float32)
    used = O.delayed_scale_run(amax, interval, hist, 12)
    state = torch.empty(H.SCALE_STATE_BYTES, dtype=torch.uint8, device="cuda")
    H.hif8_scale_state_init(state, hist)
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    for t in range(T):
        H.hif8_delayed_scale_encode(to_dev(tensors[t]), dtype, out, n, rnd, 0, 0, state, t % interval == 0, 12)
        ref = O.encode(tensors[t], dtype, int(used[t]), rnd, quick=True)
        assert np.array_equal(out.cpu().numpy(), ref), f"iteration {t}"
        words = state[:32].cpu().numpy().view(np.int32)
        expect_next = used[t + 1] if t + 1 < T else None
        if expect_next is not None:
            assert words[0] == expect_next, f"exponent after iteration {t}"
        if t % interval == 0:
            assert state[16:20].cpu().numpy().view(np.float32)[0] == amax[t]


def test_delayed_scale_argument_checks():
    state = torch.empty(H.SCALE_STATE_BYTES + 256, dtype=torch.uint8, device="cuda")
    base = state.data_ptr()
    aligned = (base + 255) // 256 * 256
    assert H.hif8_scale_state_init(aligned + 4, 1, check=False) == 8
    assert H.hif8_scale_state_init(aligned, 0, check=False) == 6
    assert H.hif8_scale_state_init(aligned, H.SCALE_HISTORY_MAX + 1, check=False) == 6
    assert H.hif8_scale_state_init(aligned, H.SCALE_HISTORY_MAX) == 0
    x = torch.ones(8, device="cuda")
    out = torch.empty(8, dtype=torch.uint8, device="cuda")
    assert H.hif8_delayed_scale_encode(x, H.F32, out, 8, H.RND_TA, 0, 0, None, 1, check=False) == 1
    assert H.hif8_delayed_scale_encode(x, H.F32, out, 8, H.RND_TA, 0, 0, aligned, 1, target_exp=16, check=False) == 5
    assert H.hif8_delayed_scale_encode(x, H.F32, out, 0, H.RND_TA, 0, 0, aligned, 1) == 0
