"""Pins for the oracle's per-channel weight scaling (Section 5.1: per-tensor scaling for activations and per-channel
scaling for weights) and for the every-N-iterations amax cadence of Section 5.1.  Each check compares the oracle
with something it does not compute itself: the already pinned per-tensor routines on extracted slices, properties
that hold for any correct implementation, or sequences worked out by hand."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import hif8_oracle as O


def weight(rows, cols, seed, dtype):
    x = W.normal_f32(rows * cols, seed).reshape(rows, cols)
    x *= np.exp2(np.random.default_rng(seed).integers(-12, 12, size=(1, cols))).astype(np.float32)  # channels differ
    x[3, 5] = np.inf
    x[4, 7] = np.nan
    x[:, 2] = 0.0  # an all-zero column
    return x if dtype == O.F32 else W.f32_to_bf16_bits(x)


@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
@pytest.mark.parametrize("axis", [0, 1])
def test_channel_scale_is_the_per_tensor_rule_on_each_slice(dtype, axis):
    x = weight(37, 29, 11, dtype)
    amax, se = O.channel_amax_scale(x, dtype, axis, target_exp=9)
    for c in range(x.shape[axis]):
        sl = np.ascontiguousarray(x[c, :] if axis == 0 else x[:, c])
        a1, s1 = O.amax_scale(sl, dtype, 9)  # pinned in test_oracle_pins.py::test_amax_scale_closed_form
        assert (amax[c], se[c]) == (np.float32(a1), s1)
        if a1 > 0:
            assert 2.0 ** 9 <= a1 * 2.0 ** s1 < 2.0 ** 10
    if axis == 1:
        assert amax[2] == 0 and se[2] == 0  # the all-zero column keeps exponent 0


@pytest.mark.parametrize("mode", [O.TA, O.HR, O.SR])
@pytest.mark.parametrize("axis", [0, 1])
def test_channel_encode_against_slices_transpose_and_uniform_case(mode, axis):
    dtype = O.BF16
    x = weight(24, 40, 5, dtype)
    _, se = O.channel_amax_scale(x, dtype, axis)
    q = O.channel_encode(x, dtype, axis, se, rnd=mode, seed=9)
    if mode != O.SR:
        # deterministic given the source bits: every channel equals the flat encoder on that slice ...
        for c in range(x.shape[axis]):
            sl = np.ascontiguousarray(x[c, :] if axis == 0 else x[:, c])
            assert np.array_equal(q[c, :] if axis == 0 else q[:, c], O.encode(sl, dtype, int(se[c]), mode))
        # ... and the transposed matrix with the other axis gives the transposed codes
        qt = O.channel_encode(np.ascontiguousarray(x.T), dtype, 1 - axis, se, rnd=mode)
        assert np.array_equal(qt.T, q)
    # one common exponent: the flat per-tensor encoder, stochastic words included (flat index r * cols + c)
    same = np.full(x.shape[axis], 3, dtype=np.int32)
    assert np.array_equal(O.channel_encode(x, dtype, axis, same, rnd=mode, seed=9).ravel(),
                          O.encode(x.ravel(), dtype, 3, mode, seed=9))


def test_channel_scale_shift_property():
    # multiplying one channel by 2^j moves that channel's exponent by -j and changes no code anywhere
    x = W.normal_f32(32 * 16, 3).reshape(32, 16)
    _, se = O.channel_amax_scale(x, O.F32, 1)
    q = O.channel_encode(x, O.F32, 1, se)
    y = x.copy()
    y[:, 4] *= 2.0 ** 7
    _, se2 = O.channel_amax_scale(y, O.F32, 1)
    d = se2 - se
    assert d[4] == -7 and not d[np.arange(16) != 4].any()
    assert np.array_equal(O.channel_encode(y, O.F32, 1, se2), q)


def test_channel_roundtrip_error_bound():
    # TA keeps >= 1 mantissa bit over the whole normal range: |w - dec| <= 2^-2 |w| at worst, 2^-4 |w| near amax
    x = W.normal_f32(64 * 48, 8).reshape(64, 48) * np.exp2(np.arange(48) - 24).astype(np.float32)
    _, se = O.channel_amax_scale(x, O.F32, 1, 14)
    q = O.channel_encode(x, O.F32, 1, se)
    back = np.stack([O.decode(q[:, c], O.F32, int(se[c])).view(np.float32) for c in range(48)], axis=1).astype(np.float64)
    big = np.abs(x) * np.exp2(se)[None, :] >= 2.0 ** -15
    assert np.all(np.abs(back - x)[big] <= 2.0 ** -2 * np.abs(x)[big])
    top = np.abs(x) * np.exp2(se)[None, :] >= 2.0 ** 8       # scaled exponent in [8, 15]: 1 or 2 mantissa bits
    assert np.all(np.abs(back - x)[top] <= 2.0 ** -2 * np.abs(x)[top])
    mid = (np.abs(x) * np.exp2(se)[None, :] >= 2.0 ** -3) & (np.abs(x) * np.exp2(se)[None, :] < 2.0 ** 3)
    assert mid.any() and np.all(np.abs(back - x)[mid] <= 2.0 ** -4 * np.abs(x)[mid] * (1 + 1e-12))


@pytest.mark.parametrize("w_is_nk", [0, 1])
def test_gemm_channel_is_the_per_tensor_product_times_column_powers(w_is_nk):
    M, N, K = 9, 12, 48
    Aq = W.random_codes(M * K, 1).reshape(M, K)
    Wq = W.random_codes(K * N, 2).reshape((N, K) if w_is_nk else (K, N))
    for t in (Aq, Wq):
        t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x10
    sw = np.random.default_rng(4).integers(-20, 20, size=N).astype(np.int32)
    rows, cols = np.divmod(np.arange(M * N), N)
    c0, s0 = O.gemm_entries(Aq, Wq, w_is_nk, 0, 0, rows, cols)  # pinned against numpy in test_oracle_pins.py
    c1, s1 = O.gemm_entries_channel(Aq, Wq, w_is_nk, 5, sw, rows, cols)
    f = np.exp2(-(5.0 + sw[cols]))
    assert np.array_equal(c1, c0 * f) and np.array_equal(s1, s0 * f)
    # a column's exponent must not leak into its neighbours
    sw2 = sw.copy()
    sw2[3] += 1
    c2, _ = O.gemm_entries_channel(Aq, Wq, w_is_nk, 5, sw2, rows, cols)
    assert np.array_equal(c2[cols != 3], c1[cols != 3]) and np.array_equal(c2[cols == 3] * 2, c1[cols == 3])


def test_delayed_scale_sequences_worked_by_hand():
    # history of one, update every iteration: iteration t uses the exponent of the amax seen at t-1; the first uses 0
    amax = np.array([3.0, 0.4, 100.0, 100.0, 0.0, 7.0], dtype=np.float32)
    #    floor(log2):   1    -2     6      6     -    2         target 14 ->  13, 16, 8, 8, 0(amax 0), 12
    assert O.delayed_scale_run(amax, 1, 1, 14).tolist() == [0, 13, 16, 8, 8, 0]
    # history of three: the exponent follows the largest of the last three measurements
    #   rings: [3] [3,.4] [3,.4,100] [.4,100,100] [100,100,0] [100,0,7]   max: 3 3 100 100 100 100
    assert O.delayed_scale_run(amax, 1, 3, 14).tolist() == [0, 13, 13, 8, 8, 8]
    # a spike leaves the ring after hist_len further measurements
    spike = np.array([1, 1, 64, 1, 1, 1, 1], dtype=np.float32)
    assert O.delayed_scale_run(spike, 1, 2, 14).tolist() == [0, 14, 14, 8, 8, 14, 14]
    # measurements only at multiples of the interval; values in between are never read
    seq = np.array([2.0, 999, 999, 0.5, 999, 999, 32.0, 999], dtype=np.float32)
    assert O.delayed_scale_run(seq, 3, 1, 10).tolist() == [0, 9, 9, 9, 11, 11, 11, 5]


def test_delayed_scale_with_history_one_matches_the_per_tensor_rule():
    rng = np.random.default_rng(2)
    tensors = [W.normal_f32(257, 100 + t) * np.float32(2.0 ** rng.integers(-30, 30)) for t in range(12)]
    amax = np.array([np.max(np.abs(x)) for x in tensors], dtype=np.float32)
    used = O.delayed_scale_run(amax, 1, 1, 12)
    assert used[0] == 0
    for t in range(1, 12):
        assert used[t] == O.amax_scale(tensors[t - 1], O.F32, 12)[1]


# ----------------------------------------------------------------------------- backward-pass operand forms
@pytest.mark.parametrize("mode", [O.TA, O.HR, O.SR])
def test_encode_transpose_is_the_flat_encoder_followed_by_a_transpose(mode):
    x = W.f32_to_bf16_bits(W.normal_f32(33 * 20, 6).reshape(33, 20) * np.float32(300.0))
    q = O.encode(x.ravel(), O.BF16, -2, mode, seed=4).reshape(33, 20)   # pinned flat encoder, source-order words
    qt = O.encode_transpose(x, O.BF16, -2, mode, seed=4)
    assert qt.shape == (20, 33) and np.array_equal(qt, q.T)
    if mode != O.SR:  # deterministic modes: transposing twice is the identity on the codes' values
        back = O.decode(qt, O.BF16, -2)
        assert np.array_equal(O.encode_transpose(back, O.BF16, -2, O.TA), q)


def test_gemm_ex_equals_the_plain_gemm_on_explicitly_transposed_operands():
    M, N, K = 7, 10, 32
    A = W.random_codes(M * K, 11).reshape(M, K)
    Wk = W.random_codes(K * N, 12).reshape(K, N)
    for t in (A, Wk):
        t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x21
    rows, cols = np.divmod(np.arange(M * N), N)
    ref = O.gemm_entries(A, Wk, 0, 3, -2, rows, cols)  # pinned against numpy in test_oracle_pins.py
    for a_km in (0, 1):
        for w_nk in (0, 1):
            got = O.gemm_entries_ex(np.ascontiguousarray(A.T) if a_km else A, a_km,
                                    np.ascontiguousarray(Wk.T) if w_nk else Wk, w_nk, 3, -2, rows, cols)
            assert np.array_equal(got[0], ref[0]) and np.array_equal(got[1], ref[1])
    sw = np.arange(N, dtype=np.int32) - 4
    ch = O.gemm_entries_ex(np.ascontiguousarray(A.T), 1, Wk, 0, 3, sw, rows, cols)
    ref_ch = O.gemm_entries_channel(A, Wk, 0, 3, sw, rows, cols)
    assert np.array_equal(ch[0], ref_ch[0]) and np.array_equal(ch[1], ref_ch[1])
    # a non-square case where a wrong leading dimension or swapped index cannot cancel: one-hot operands
    A1 = np.zeros((M, K), dtype=np.uint8); A1[2, 5] = 0x08          # value 1 at (m=2, k=5)
    W1 = np.zeros((K, N), dtype=np.uint8); W1[5, 7] = 0x10          # value 2 at (k=5, n=7)
    c, _ = O.gemm_entries_ex(np.ascontiguousarray(A1.T), 1, np.ascontiguousarray(W1.T), 1, 0, 0, rows, cols)
    expect = np.zeros(M * N); expect[2 * N + 7] = 2.0
    assert np.array_equal(c, expect)


# ----------------------------------------------------------------------------- adaptive loss scaling (Section 5.1)
def test_als_initial_state_and_window_walk_worked_by_hand():
    # the paper's start: scale 2^32, window 20.  60 clean iterations = three increases -> window 50
    se, win = O.als_run(np.zeros(60 + 150 + 1, dtype=np.int32))
    assert se[0] == 32 and win[0] == 20
    assert se[19] == 32 and se[20] == 33 and se[40] == 34 and se[60] == 35   # an increase after every 20 clean steps
    assert win[59] == 20 and win[60] == 50                                      # third increase moves the window up
    assert se[60 + 49] == 35 and se[60 + 50] == 36 and se[60 + 100] == 37 and se[60 + 150] == 38
    assert win[60 + 149] == 50 and win[60 + 150] == 100
    # three overflows in a row: three halvings, then the window steps down the list (20 -> 1)
    se, win = O.als_run(np.array([1, 1, 1, 0, 0, 0, 0], dtype=np.int32))
    assert se.tolist() == [32, 31, 30, 29, 30, 31, 32] and win.tolist() == [20, 20, 20, 1, 1, 1, 20]
    # (with window 1 every clean step doubles, so the third clean step is the third increase: back up to 20)
    se, win = O.als_run(np.array([1, 1, 1, 0, 0, 0, 0, 0], dtype=np.int32))
    assert win.tolist() == [20, 20, 20, 1, 1, 1, 20, 20] and se[7] == 32 and se[6] == 32
    # an increase between overflows breaks the run of decreases: two overflows, 20 clean steps (one increase), one more
    f = np.array([1, 1] + [0] * 20 + [1, 0], dtype=np.int32)
    se, win = O.als_run(f)
    assert np.all(win == 20) and se[22] == 31 and se[23] == 30
    # clean steps that do not change the scale do not break it (window 20: 5 clean steps change nothing)
    f = np.array([1] + [0] * 5 + [1] + [0] * 5 + [1, 0], dtype=np.int32)
    se, win = O.als_run(f)
    assert win[12] == 20 and win[13] == 1 and se[13] == 29
    # the list ends: the window stays at 1 / at 1000
    se, win = O.als_run(np.ones(40, dtype=np.int32), init_window_index=0)
    assert np.all(win == 1) and se[39] == 32 - 39
    se, win = O.als_run(np.zeros(1000 * 7, dtype=np.int32), init_window_index=6)
    assert np.all(win == 1000) and se[-1] == 32 + 6
    assert O.ALS_WINDOWS == (1, 20, 50, 100, 200, 500, 1000)


def test_als_scale_rule_against_the_library_loss_scaler():
    # given the oracle's windows, the scale must follow torch's dynamic loss-scale update (growth 2, backoff 1/2)
    rng = np.random.default_rng(7)
    f = (rng.random(4000) < 0.02).astype(np.int32)
    f[100:103] = 1
    f[900:906] = 1
    se, win = O.als_run(f, init_scale_exp=16)
    scale = torch.tensor(2.0 ** 16)
    tracker = torch.tensor(0, dtype=torch.int32)
    for t in range(f.size):
        assert float(scale) == 2.0 ** int(se[t]), t
        torch._amp_update_scale_(scale, tracker, torch.tensor(float(f[t])), 2.0, 0.5, int(win[t]))
    assert len(set(win.tolist())) >= 3      # the walk visited several windows
