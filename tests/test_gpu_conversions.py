"""GPU parity: every conversion entry point, through the C ABI, bit-exact against the CPU oracle."""
import numpy as np
import pytest
import torch

import paper_2409_16626_b200 as H
import workloads as W
from oracle import hif8_oracle as O

from gpu_util import NP_OF, dev_empty, to_dev, workspace

pytestmark = pytest.mark.gpu

MODES = [H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR]
FLAGSETS = [0, H.FLAG_SATURATE, H.FLAG_NAN_TO_ZERO, H.FLAG_SATURATE | H.FLAG_NAN_TO_ZERO]


def gpu_encode(src_bits, dtype, offset_in=0, offset_out=0, **kw):
    n = src_bits.size
    if offset_in:
        item = src_bits.dtype.itemsize
        raw = torch.empty(n * item + offset_in + 16, dtype=torch.uint8, device="cuda")
        raw[offset_in:offset_in + n * item] = torch.from_numpy(src_bits.view(np.uint8).copy()).cuda()
        src_ptr, keep = raw.data_ptr() + offset_in, raw
    else:
        keep = to_dev(src_bits)
        src_ptr = keep.data_ptr()
    _, dptr, rb = dev_empty(n, np.uint8, offset_out)
    H.hif8_encode(src_ptr, dtype, dptr, n, **kw)
    torch.cuda.synchronize()
    return rb()


def assert_same(got, want, src=None):
    if not np.array_equal(got, want):
        bad = np.nonzero(got != want)[0]
        i = bad[0]
        msg = f"{bad.size} mismatches; first at {i}: got {got[i]:#x} want {want[i]:#x}"
        if src is not None:
            msg += f" src {src.reshape(-1)[i]:#x}"
        raise AssertionError(msg)


# ----------------------------------------------------------------------------- decode
@pytest.mark.parametrize("dtype", [H.F32, H.BF16, H.F16])
@pytest.mark.parametrize("scale_exp", [0, 5, -7, 126, -126, 20, -20])
def test_decode_all_codes(dtype, scale_exp):
    codes = np.tile(np.arange(256, dtype=np.uint8), 37)[: 256 * 37 - 5]      # several tiles and a ragged tail
    d = to_dev(codes)
    _, ptr, rb = dev_empty(codes.size, NP_OF[dtype])
    H.hif8_decode(d, ptr, dtype, codes.size, scale_exp)
    torch.cuda.synchronize()
    assert_same(rb(), O.decode(codes, dtype, scale_exp))


@pytest.mark.parametrize("dtype", [H.F32, H.BF16, H.F16])
def test_decode_large_random_and_misaligned(dtype):
    codes = W.random_codes(3_000_011, seed=21, finite_only=False)
    want = O.decode(codes, dtype, 3)
    for off_in, off_out in [(0, 0), (3, 0), (0, 4), (1, 2)]:
        raw = torch.empty(codes.size + 32, dtype=torch.uint8, device="cuda")
        raw[off_in:off_in + codes.size] = torch.from_numpy(codes).cuda()
        item = np.dtype(NP_OF[dtype]).itemsize
        _, ptr, rb = dev_empty(codes.size, NP_OF[dtype], off_out * item if off_out else 0)
        H.hif8_decode(raw.data_ptr() + off_in, ptr, dtype, codes.size, 3)
        torch.cuda.synchronize()
        assert_same(rb(), want)


# ----------------------------------------------------------------------------- encode, exhaustive 16-bit
@pytest.mark.parametrize("dtype", [H.BF16, H.F16])
@pytest.mark.parametrize("mode", MODES)
def test_encode_exhaustive_16bit(dtype, mode):
    bits = W.all_u16()
    for flags in FLAGSETS:
        want = O.encode(bits, dtype, 0, mode, flags, seed=1, quick=False)
        assert_same(gpu_encode(bits, dtype, scale_exp=0, rnd=mode, flags=flags, seed=1), want, bits)
    for se in (3, -9, 14, -30, 100, -100, 126, 110):  # the last two bring subnormal BF16 sources into range
        want = O.encode(bits, dtype, se, mode, 0, seed=7, quick=True)
        assert_same(gpu_encode(bits, dtype, scale_exp=se, rnd=mode, seed=7), want, bits)


# ----------------------------------------------------------------------------- encode, FP32
def f32_cases():
    special = np.array([0x00000000, 0x80000000, 0x7F800000, 0xFF800000, 0x7FC00000, 0xFFC00000, 0x7F800001,
                        0xFF800001, 0x7FFFFFFF, 0x00000001, 0x807FFFFF, 0x00800000, 0x7F7FFFFF, 0x47200000,
                        0x471FFFFF, 0x47400000, 0x473FFFFF, 0x34000000, 0x33FFFFFF, 0x34800000, 0x347FFFFF],
                       dtype=np.uint32)
    return {
        "normal": W.normal_f32(1_000_003, seed=1234).view(np.uint32),
        "loguniform": W.loguniform_f32(1_000_003, seed=3456).view(np.uint32),
        "bits": np.concatenate([special, W.random_bits_f32(500_000, seed=9).view(np.uint32)]),
    }


@pytest.mark.parametrize("mode", MODES)
def test_encode_f32(mode):
    for name, bits in f32_cases().items():
        for se, flags in [(0, 0), (0, 3), (7, 0), (-5, 1), (126, 0), (-126, 2), (110, 0)]:
            want = O.encode(bits, O.F32, se, mode, flags, seed=42, quick=True)
            got = gpu_encode(bits, H.F32, scale_exp=se, rnd=mode, flags=flags, seed=42)
            assert_same(got, want, bits)


def test_encode_f32_subnormal_sources_with_large_scale():
    bits = np.concatenate([np.arange(1, 1 << 16, dtype=np.uint32), (np.arange(1 << 12, dtype=np.uint32) << 11) | 0x400,
                           np.arange(0x7F0000, 0x810000, dtype=np.uint32)])
    bits = np.concatenate([bits, bits | 0x80000000]).astype(np.uint32)
    for mode in MODES:
        for se in (126, 120, 104, 103):
            want = O.encode(bits, O.F32, se, mode, 0, seed=3, quick=True)
            assert_same(gpu_encode(bits, H.F32, scale_exp=se, rnd=mode, seed=3), want, bits)


@pytest.mark.parametrize("mode", [H.RND_TA, H.RND_SR, H.RND_HR, H.RND_SSR])
def test_encode_ragged_sizes_and_misaligned_pointers(mode):
    base = W.loguniform_f32(5000, seed=5, lo_exp=-26, hi_exp=17).view(np.uint32)
    for n in (1, 3, 4, 15, 16, 17, 1023, 1024, 1025, 4097):
        bits = base[:n]
        want = O.encode(bits, O.F32, 0, mode, 0, seed=11, quick=True)
        for off_in, off_out in [(0, 0), (4, 0), (0, 1), (8, 3)]:
            assert_same(gpu_encode(bits, H.F32, offset_in=off_in, offset_out=off_out, rnd=mode, seed=11), want)
    b16 = W.normal_bf16(4099, seed=6)
    want = O.encode(b16, O.BF16, 2, mode, 0, seed=11, quick=True)
    for off_in, off_out in [(0, 0), (2, 0), (0, 5), (6, 1)]:
        assert_same(gpu_encode(b16, H.BF16, offset_in=off_in, offset_out=off_out, scale_exp=2, rnd=mode, seed=11), want)
    assert H.hif8_encode(0, H.F32, 0, 0) == 0


def test_encode_sizes_around_the_groups_per_block_steps():
    # Large tensors give a block two, three or four groups of vectors (grid-stride) and skip the bounds checks of groups
    # that lie wholly inside the tensor: sizes just below and above each step, with ragged vector and element tails,
    # every element compared
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    wave, per_group = sms * 8, 256 * 4 * 4                    # resident blocks per wave; FP32 elements per group
    base = W.loguniform_f32(1 << 22, seed=77, lo_exp=-26, hi_exp=17).view(np.uint32)
    for groups in (2, 3, 4):
        for n in (groups * wave * per_group - 4099, groups * wave * per_group + 3 * per_group + 1027):
            bits = np.resize(base, n)
            d_src = to_dev(bits)
            for mode in (H.RND_TA, H.RND_HR) + ((H.RND_SR,) if groups == 2 else ()):
                _, dptr, rb = dev_empty(n, np.uint8)
                H.hif8_encode(d_src, H.F32, dptr, n, 3, mode, 0, 21)
                torch.cuda.synchronize()
                assert np.array_equal(rb(), O.encode(bits, O.F32, 3, mode, 0, seed=21, quick=True))
    # the BF16 fake-quant kernels (rounding on the bit pattern) take the same grid rule
    n = 4 * wave * 256 * 4 * 8 + 8 * 1024 + 13
    b16 = np.resize(W.llm_activation_bf16(512, 4096, seed=5).reshape(-1), n)
    d = to_dev(b16)
    for mode in (H.RND_TA, H.RND_HR):
        _, dptr, rb = dev_empty(n, np.uint16)
        H.hif8_fake_quant(d, dptr, H.BF16, n, 0, 4, mode, 0, 9)
        torch.cuda.synchronize()
        assert np.array_equal(rb(), O.fake_quant(b16, O.BF16, 4, mode, 0, seed=9, quick=True))


def test_encode_sr_index_is_the_element_offset():
    # the threshold of element i depends on (seed, i) only: a long tensor and a slice of it differ
    bits = np.full(100_000, np.float32(1.03).view(np.uint32), dtype=np.uint32)
    full = gpu_encode(bits, H.F32, rnd=H.RND_SR, seed=5)
    assert_same(full, O.encode(bits, O.F32, 0, O.SR, 0, seed=5, quick=True))
    assert 0.2 < np.mean(full == full.max()) < 0.3          # F = 0.24
    other = gpu_encode(bits, H.F32, rnd=H.RND_SR, seed=6)
    assert np.any(other != full)


# ----------------------------------------------------------------------------- amax + scale + encode
@pytest.mark.parametrize("dtype", [H.F32, H.BF16, H.F16])
def test_amax_scale_encode_jit_and_delayed(dtype):
    n = 2_000_003
    if dtype == H.F32:
        src = W.normal_f32(n, seed=1234).view(np.uint32).copy()
        src[[5, 77]] = [0x7F800000, 0x7FC00000]              # Inf / NaN do not take part in amax
    elif dtype == H.BF16:
        src = W.llm_activation_bf16(n // 1000 + 1, 1000, seed=2345).reshape(-1)[:n].copy()
        src[[5, 77]] = [0x7F80, 0x7FC1]
    else:
        src = W.normal_f32(n, seed=77, std=3.0).astype(np.float16).view(np.uint16).copy()
        src[[5, 77]] = [0xFC00, 0x7E01]
    ws, wsb = workspace()
    d_src = to_dev(src)
    outs = torch.zeros(4, dtype=torch.int32, device="cuda")
    for target in (14, 3):
        amax, se = O.amax_scale(src, dtype, target)
        for mode in (H.RND_TA, H.RND_HR):
            _, dptr, rb = dev_empty(n, np.uint8)
            H.hif8_amax_scale_encode(d_src, dtype, dptr, n, target, mode, 0, 0, None, outs[0:1], outs[1:2], outs[2:3],
                                     ws, wsb)
            torch.cuda.synchronize()
            o = outs.cpu().numpy()
            assert o[0:1].view(np.float32)[0] == np.float32(amax) and o[1] == se
            assert o[2:3].view(np.float32)[0] == np.float32(2.0) ** se
            assert_same(rb(), O.encode(src, dtype, se, mode, 0, quick=True), src)
    # delayed scaling: exponent given on the device, amax of this tensor still reported
    amax, _ = O.amax_scale(src, dtype, 14)
    d_se = torch.tensor([5], dtype=torch.int32, device="cuda")
    outs.zero_()
    _, dptr, rb = dev_empty(n, np.uint8)
    H.hif8_amax_scale_encode(d_src, dtype, dptr, n, 14, H.RND_TA, 0, 0, d_se, outs[0:1], outs[1:2], outs[2:3], ws, wsb)
    torch.cuda.synchronize()
    o = outs.cpu().numpy()
    assert o[0:1].view(np.float32)[0] == np.float32(amax) and o[1] == 5 and o[2:3].view(np.float32)[0] == 32.0
    assert_same(rb(), O.encode(src, dtype, 5, O.TA, 0, quick=True), src)


def test_amax_alone():
    ws, wsb = workspace()
    out = torch.zeros(1, dtype=torch.float32, device="cuda")
    for dtype, src in [(H.F32, W.loguniform_f32(1_000_003, seed=4).view(np.uint32)), (H.BF16, W.normal_bf16(300_001, seed=5)),
                       (H.F16, W.normal_f32(70_001, seed=6).astype(np.float16).view(np.uint16)),
                       (H.F32, np.array([0x7FC00000, 0xFF800000, 0x80000000], np.uint32))]:
        for _ in range(2):
            H.hif8_amax(to_dev(src), dtype, src.size, out, ws, wsb)
            torch.cuda.synchronize()
            assert float(out.item()) == O.amax_scale(src, dtype, 14)[0]


def test_amax_degenerate_tensors():
    ws, wsb = workspace()
    outs = torch.zeros(4, dtype=torch.int32, device="cuda")
    for src, want_se in [(np.zeros(1000, np.uint32), 0), (np.full(999, 0x7FC00000, np.uint32), 0),
                         (np.full(17, 0x00000003, np.uint32), 126), (np.full(5, 0x7F7FFFFF, np.uint32), 14 - 127)]:
        amax, se = O.amax_scale(src, O.F32, 14)
        assert se == want_se
        _, dptr, rb = dev_empty(src.size, np.uint8)
        H.hif8_amax_scale_encode(to_dev(src), H.F32, dptr, src.size, 14, H.RND_TA, 0, 0, None, outs[0:1], outs[1:2], None,
                                 ws, wsb)
        torch.cuda.synchronize()
        o = outs.cpu().numpy()
        assert o[0:1].view(np.float32)[0] == np.float32(amax) and o[1] == se
        assert_same(rb(), O.encode(src, O.F32, se, O.TA, 0, quick=True))


# ----------------------------------------------------------------------------- fake-quant
@pytest.mark.parametrize("dtype", [H.F32, H.BF16, H.F16])
@pytest.mark.parametrize("mode", MODES)
def test_fake_quant(dtype, mode):
    n = 300_007
    if dtype == H.F32:
        src = np.concatenate([W.loguniform_f32(n, seed=8, lo_exp=-30, hi_exp=20).view(np.uint32),
                              W.random_bits_f32(20_000, seed=10).view(np.uint32)])
    elif dtype == H.BF16:
        src = np.concatenate([W.llm_activation_bf16(301, 1000, seed=2345).reshape(-1), W.all_u16()])
    else:
        src = np.concatenate([W.normal_f32(n, seed=8).astype(np.float16).view(np.uint16), W.all_u16()])
    d_src = to_dev(src)
    for se, flags in [(0, 0), (6, 3), (-3, 0), (125, 0), (-125, 0)]:
        _, dptr, rb = dev_empty(src.size, NP_OF[dtype])
        H.hif8_fake_quant(d_src, dptr, dtype, src.size, 0, se, mode, flags, 9)
        torch.cuda.synchronize()
        assert_same(rb(), O.fake_quant(src, dtype, se, mode, flags, seed=9, quick=True), src)
    # fused amax, in place
    ws, wsb = workspace()
    outs = torch.zeros(2, dtype=torch.int32, device="cuda")
    amax, se = O.amax_scale(src, dtype, 14)
    buf = d_src.clone()
    H.hif8_fake_quant(buf, buf, dtype, src.size, 1, 14, mode, 0, 9, outs[0:1], outs[1:2], ws, wsb)
    torch.cuda.synchronize()
    o = outs.cpu().numpy()
    assert o[0:1].view(np.float32)[0] == np.float32(amax) and o[1] == se
    got = buf.cpu().numpy().view(NP_OF[dtype])
    assert_same(got, O.fake_quant(src, dtype, se, mode, 0, seed=9, quick=True), src)


def test_fake_quant_bf16_standard_sr_many_thresholds_per_pattern():
    # the in-place kernel's standard SR: every BF16 pattern at 32 positions (32 different Philox words each), several
    # scales and seeds, both options; the last positions run through the scalar tail
    src = np.tile(W.all_u16(), 32)[:-3]
    d_src = to_dev(src)
    for se, flags, seed in [(0, 0, 1), (5, 3, 2), (-20, 0, 3), (14, 1, 0xDEADBEEF12345678), (30, 2, 5)]:
        _, dptr, rb = dev_empty(src.size, np.uint16)
        H.hif8_fake_quant(d_src, dptr, H.BF16, src.size, 0, se, H.RND_SR, flags, seed)
        torch.cuda.synchronize()
        assert_same(rb(), O.fake_quant(src, O.BF16, se, O.SR, flags, seed=seed, quick=True), src)


@pytest.mark.parametrize("mode,omode", [(H.RND_TA, O.TA), (H.RND_TE, O.TE), (H.RND_HR, O.HR), (H.RND_SSR, O.SSR), (H.RND_SR, O.SR)])
def test_fake_quant_bf16_in_place_scale_edges_and_tails(mode, omode):
    # the in-place kernel rounds BF16 with per-exponent constants (packed BF16 arithmetic except for round half away):
    # scales at which a constant leaves the BF16 range or subnormal sources come into range, every pattern; then ragged,
    # misaligned pieces
    src = W.all_u16()
    d_src = to_dev(src)
    for se in (14, -30, 100, 101, 104, 111, 112, 120, 122, 126, -100, -105, -110, -120, -126):
        _, dptr, rb = dev_empty(src.size, np.uint16)
        H.hif8_fake_quant(d_src, dptr, H.BF16, src.size, 0, se, mode, 0, 0)
        torch.cuda.synchronize()
        assert_same(rb(), O.fake_quant(src, O.BF16, se, omode, 0, quick=True), src)
    part = W.llm_activation_bf16(7, 1000, seed=5).reshape(-1)
    for n, off in [(1, 0), (7, 0), (8, 0), (9, 2), (1025, 0), (4099, 6), (6999, 2)]:
        piece = part[:n]
        raw = torch.zeros(2 * n + 32, dtype=torch.uint8, device="cuda")
        raw[off:off + 2 * n] = torch.from_numpy(piece.view(np.uint8).copy()).cuda()
        out = torch.zeros(2 * n + 32, dtype=torch.uint8, device="cuda")
        H.hif8_fake_quant(raw.data_ptr() + off, out.data_ptr() + off, H.BF16, n, 0, 5, mode, 3, 0)
        torch.cuda.synchronize()
        got = out[off:off + 2 * n].cpu().numpy().view(np.uint16)
        assert_same(got, O.fake_quant(piece, O.BF16, 5, omode, 3, quick=True), piece)


# ----------------------------------------------------------------------------- full sizes: sampled outputs
def test_config2_full_size():
    # FP32 4096x4096 N(0,1): per-tensor scaled encode + decode, every element (neighbour-pair oracle), and a strided
    # sample plus both ends through the oracle's scan of all 256 codes
    x = W.normal_f32((4096, 4096), seed=1234).reshape(-1)
    n = x.size
    ws, wsb = workspace()
    outs = torch.zeros(4, dtype=torch.int32, device="cuda")
    d_src = to_dev(x)
    codes = torch.empty(n, dtype=torch.uint8, device="cuda")
    back = torch.empty(n, dtype=torch.int32, device="cuda")
    H.hif8_amax_scale_encode(d_src, H.F32, codes, n, 14, H.RND_TA, 0, 0, None, outs[0:1], outs[1:2], outs[2:3], ws, wsb)
    torch.cuda.synchronize()
    amax, se = O.amax_scale(x, O.F32, 14)
    assert int(outs[1]) == se
    H.hif8_decode(codes, back, H.F32, n, se)
    torch.cuda.synchronize()
    got_codes = codes.cpu().numpy()
    want_codes = O.encode(x, O.F32, se, O.TA, 0, quick=True)
    assert_same(got_codes, want_codes)
    assert_same(back.cpu().numpy().view(np.uint32), O.decode(want_codes, O.F32, se))
    idx = np.unique(np.concatenate([np.arange(0, n, 53), np.arange(0, 70000), np.arange(n - 70000, n)]))
    assert_same(got_codes[idx], O.encode(x[idx], O.F32, se, O.TA, 0, quick=False))


def test_f32_full_sweep_all_2_32_patterns():
    # every FP32 encoding, unscaled, round-half-away: 64 slices of 2^26 patterns generated from the index
    n = 1 << 26
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    ar = torch.arange(n, dtype=torch.int64, device="cuda")
    for chunk in range(64):
        first = chunk << 26
        d = (ar + first).to(torch.int32) if first < (1 << 31) else (ar + (first - (1 << 32))).to(torch.int32)
        H.hif8_encode(d, H.F32, out, n, 0, H.RND_TA)
        torch.cuda.synchronize()
        want = O.encode_f32_range(first, n, 0, O.TA, 0, 0, quick=True)
        got = out.cpu().numpy()
        if not np.array_equal(got, want):
            i = int(np.nonzero(got != want)[0][0])
            raise AssertionError(f"pattern {first + i:#010x}: got {got[i]:#x} want {want[i]:#x}")


@pytest.mark.parametrize("mode", [H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR])
def test_f32_full_sweep_other_modes(mode):
    # every FP32 encoding of either sign in every other rounding mode, 64 slices of 2^26 patterns
    n = 1 << 26
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    ar = torch.arange(n, dtype=torch.int64, device="cuda")
    for chunk in range(64):
        first = chunk << 26
        d = (ar + first).to(torch.int32) if first < (1 << 31) else (ar + (first - (1 << 32))).to(torch.int32)
        H.hif8_encode(d, H.F32, out, n, 0, mode, 0, 77)
        torch.cuda.synchronize()
        want = O.encode_f32_range(first, n, 0, mode, 0, 77, quick=True)
        got = out.cpu().numpy()
        if not np.array_equal(got, want):
            i = int(np.nonzero(got != want)[0][0])
            raise AssertionError(f"pattern {first + i:#010x}: got {got[i]:#x} want {want[i]:#x}")


@pytest.mark.parametrize("mode", [H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR])
def test_generated_f32_patterns_sweep_with_both_options(mode):
    # hif8_encode_f32_patterns: the whole FP32 range without a source tensor, here with SATURATE and NaN -> 0 switched on
    # (Section 3: the two options), against the oracle; plus equality with hif8_encode on a slice, wrap-around of the
    # pattern counter, an unaligned destination and a ragged length
    n = 1 << 26
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    omode = {H.RND_TA: O.TA, H.RND_HR: O.HR, H.RND_SSR: O.SSR, H.RND_TE: O.TE, H.RND_SR: O.SR}[mode]
    for chunk in range(64):
        first = chunk << 26
        H.hif8_encode_f32_patterns(first, out, n, 0, mode, 3, 91)
        torch.cuda.synchronize()
        want = O.encode_f32_range(first, n, 0, omode, 3, 91, quick=True)
        got = out.cpu().numpy()
        if not np.array_equal(got, want):
            i = int(np.nonzero(got != want)[0][0])
            raise AssertionError(f"pattern {first + i:#010x}: got {got[i]:#x} want {want[i]:#x}")
    first, m = 0xFFFFFF00, 1003                              # wraps through 0xFFFFFFFF -> 0, scaled, ragged, misaligned
    raw, ptr, readback = dev_empty(m, np.uint8, offset_bytes=3)
    H.hif8_encode_f32_patterns(first, ptr, m, 5, mode, 0, 7)
    bits = ((np.arange(m, dtype=np.uint64) + first) & 0xFFFFFFFF).astype(np.uint32)
    src = to_dev(bits)
    ref = torch.empty(m, dtype=torch.uint8, device="cuda")
    H.hif8_encode(src, H.F32, ref, m, 5, mode, 0, 7)
    torch.cuda.synchronize()
    assert np.array_equal(readback(), ref.cpu().numpy())
    assert np.array_equal(readback(), O.encode(bits, O.F32, 5, omode, 0, seed=7, quick=True))
