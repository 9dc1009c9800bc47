"""Pins for the CPU oracle: every check compares it with something fixed by the paper or by mathematics,
never with itself.  Citations name the paper's section / table / equation."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import workloads as W
from oracle import hif8_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MODES = [O.TA, O.HR, O.SSR, O.TE, O.SR]
DT16 = [O.BF16, O.F16]


def finite_codes():
    return [c for c in range(256) if O.parse(c)["kind"] == 1]


def pos_magnitudes():
    """Sorted positive finite magnitudes (as exact Fractions)."""
    return sorted({Fraction(O.value(c)) for c in range(128) if O.parse(c)["kind"] == 1})


def src_values(bits, dtype):
    """float64 values of 16-bit encodings through numpy library casts (not the oracle)."""
    with np.errstate(invalid="ignore"):
        if dtype == O.F16:
            return bits.view(np.float16).astype(np.float64)
        return W.bf16_bits_to_f32(bits).astype(np.float64)


# ----------------------------------------------------------------------------- format pins
def test_table4_patterns():
    for line in open(os.path.join(GOLDEN, "table4_patterns.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        pat, kind, val = line.split()
        pats = [pat.replace("S", "0"), pat.replace("S", "1")] if "S" in pat else [pat]
        for p in pats:
            c = int(p, 2)
            v = O.value(c)
            if kind == "inf":
                assert np.isinf(v) and (v < 0) == (p[0] == "1")
                assert abs(O.parse(c)["value"]) == 1.5 * 2 ** 15  # Eq. 1 value the Inf patterns replace
            elif kind == "nan":
                assert np.isnan(v)
            elif kind == "zero":
                assert v == 0.0 and not np.signbit(v)
            else:
                m, e = val.split("*2^")
                assert v == float(m) * 2.0 ** int(e), (p, v)


def test_table3_mapping_and_dot_code():
    rows = {}
    for line in open(os.path.join(GOLDEN, "table3_mapping.txt")):
        line = line.split("#")[0].strip()
        if line:
            d, code, ebits, lo, hi, w = line.split()
            rows[d] = (code, int(ebits), lo, hi, int(w))
    seen = {k: set() for k in rows}
    for c in range(256):
        f = O.parse(c)
        bits = format(c, "08b")
        key = "DML" if f["is_dml"] else str(f["D"])
        code, ebits, lo, hi, w = rows[key]
        assert bits[1:1 + len(code)] == code           # Table 2 prefix code
        assert f["w"] == w                             # Table 1 / Table 3 mantissa width
        assert 1 + len(code) + ebits + w == 8          # Table 1: the four fields fill the byte
        if key != "DML":
            assert int(lo) <= abs(f["E"]) <= int(hi)   # Table 3 exponent ranges
            seen[key].add(f["E"])
    for key, (code, ebits, lo, hi, w) in rows.items():
        if key != "DML":
            want = {e for a in range(int(lo), int(hi) + 1) for e in (a, -a)}
            assert seen[key] == want                   # every exponent reachable, through one D only


def test_abstract_counts():
    # Abstract: 7 exponents with 3-bit mantissa, 8 with 2-bit, 16 with 1-bit; 31 -> 38 binades; one zero
    by_w = {1: set(), 2: set(), 3: set()}
    nml_bin, all_bin = set(), set()
    for c in range(256):
        f = O.parse(c)
        if f["kind"] in (1, 2) and not f["is_dml"]:
            by_w[f["w"]].add(f["E"])
            nml_bin.add(f["E"])
        if f["kind"] == 1:
            all_bin.add(int(np.floor(np.log2(abs(f["value"])))))
    assert (len(by_w[3]), len(by_w[2]), len(by_w[1])) == (7, 8, 16)
    assert len(nml_bin) == 31 and len(all_bin) == 38   # also Section 2.2: 31 exponents with >= 1 mantissa bit
    assert min(nml_bin) == -15 and max(nml_bin) == 15 and min(all_bin) == -22      # Table 4 exponent rows
    assert sum(1 for c in range(256) if O.value(c) == 0.0) == 1
    assert sum(1 for c in range(256) if np.isnan(O.value(c))) == 1
    assert sum(1 for c in range(256) if np.isinf(O.value(c))) == 2


def test_non_redundancy_and_symmetry():
    vals = [O.value(c) for c in finite_codes()]
    assert len(vals) == 252 and len(set(vals)) == 252           # Section 2.2: no redundant coding
    assert len(pos_magnitudes()) == 126
    for c in range(128):
        if O.parse(c)["kind"] == 1:
            assert O.value(c | 0x80) == -O.value(c)
    for v in vals:                                              # <= 4 significant bits, Eq. 1 / Eq. 2
        m, e = np.frexp(abs(v))
        assert (m * 16) == int(m * 16) and -22 <= e - 1 <= 15


def test_equations_closed_form():
    # Eq. 1 / Eq. 2 retyped independently from the field values reported by the parser
    for c in finite_codes():
        f = O.parse(c)
        if f["is_dml"]:
            want = Fraction(2) ** (f["M"] - 23)
        else:
            want = Fraction(2) ** f["E"] * (1 + Fraction(f["M"], 2 ** f["w"]))
        assert Fraction(O.value(c)) == (-want if f["sign"] else want)
    assert [O.value(c) for c in range(1, 8)] == [2.0 ** e for e in range(-22, -15)]   # Eq. 2 range


# ----------------------------------------------------------------------------- helper formats
def test_round_to_format_matches_library_casts():
    rng = np.random.default_rng(7)
    x = np.concatenate([
        rng.standard_normal(20000) * np.exp(rng.uniform(-40, 40, 20000)),
        np.array([0.0, -0.0, np.inf, -np.inf, 65504.0, 65520.0, 65519.99, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -26,
                  2.0 ** -14, 2.0 ** -149, 2.0 ** -150, 3.4028235677973366e38, 1e39, 2.0 ** -126, 1.5 * 2 ** -133]),
    ])
    with np.errstate(over="ignore"):
        f16 = x.astype(np.float16).view(np.uint16)
        f32 = x.astype(np.float32).view(np.uint32)
    bf = (torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
    for i, v in enumerate(x):
        assert O.round_to_format(v, 5, 10) == f16[i], v
        assert O.round_to_format(v, 8, 23) == f32[i], v
        assert O.round_to_format(v, 8, 7) == bf[i], v
    assert O.round_to_format(float("nan"), 8, 23) == 0x7FC00000
    assert O.round_to_format(float("nan"), 8, 7) == 0x7FC0
    assert O.round_to_format(float("nan"), 5, 10) == 0x7E00


def test_decode_all_codes_every_dtype():
    codes = np.arange(256, dtype=np.uint8)
    want = np.array([O.value(c) for c in range(256)])
    f32 = O.decode(codes, O.F32).view(np.float32).astype(np.float64)
    f16 = O.decode(codes, O.F16).view(np.float16).astype(np.float64)
    bf = W.bf16_bits_to_f32(O.decode(codes, O.BF16)).astype(np.float64)
    for got in (f32, f16, bf):     # every HiF8 value is exact in all three formats
        assert np.array_equal(np.isnan(got), np.isnan(want))
        assert np.array_equal(got[~np.isnan(want)], want[~np.isnan(want)])
    assert not np.signbit(f32[0])
    got = O.decode(codes, O.F32, scale_exp=5).view(np.float32).astype(np.float64)   # descale: exact power of two
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok] / 32.0)


def test_philox_known_answers():
    # Known-answer vectors published with the Random123 library for philox4x32-10 (Salmon et al., SC'11)
    kat = [
        ([0, 0, 0, 0], [0, 0], [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]),
        ([0xffffffff] * 4, [0xffffffff] * 2, [0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd]),
        ([0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344], [0xa4093822, 0x299f31d0],
         [0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1]),
    ]
    for ctr, key, out in kat:
        assert [int(v) for v in O.philox4x32_10(ctr, key)] == out
    seed = 0x0123456789ABCDEF                          # element -> (counter, word) mapping
    for idx in (0, 1, 2, 3, 4, 7, 2 ** 34 + 5):
        blk = idx >> 2
        w = O.philox4x32_10([blk & 0xFFFFFFFF, blk >> 32, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert O.sr_word(seed, idx) == int(w[idx & 3])


# ----------------------------------------------------------------------------- rounding pins
def neighbours(a, mags):
    """L <= a < U among [0] + mags + [inf candidate], exact Fractions."""
    cand = [Fraction(0)] + mags + [Fraction(49152)]
    lo = max(v for v in cand if v <= a)
    hi = min(v for v in cand if v > a)
    return lo, hi


def test_te_ta_worked_example():
    # Section 3.1: three consecutive values x.1 (binary) with integer parts 00, 01, 10:
    # TE -> 00, 10, 10 ; TA -> 01, 10, 11.  Binade 2^3 has a 3-bit mantissa, spacing 1: 8.5, 9.5, 10.5.
    x = np.array([8.5, 9.5, 10.5], dtype=np.float32)
    te = [O.value(c) for c in O.encode(x, O.F32, rnd=O.TE)]
    ta = [O.value(c) for c in O.encode(x, O.F32, rnd=O.TA)]
    assert [int(v) & 3 for v in te] == [0b00, 0b10, 0b10] and te == [8.0, 10.0, 10.0]
    assert [int(v) & 3 for v in ta] == [0b01, 0b10, 0b11] and ta == [9.0, 10.0, 11.0]
    assert [O.value(c) for c in O.encode(-x, O.F32, rnd=O.TA)] == [-9.0, -10.0, -11.0]


def test_hand_cases_ta():
    cases = {2.0 ** 15: 0x6E, 2.0 ** -22: 0x01, 1.0: 0x08, -1.0: 0x88, 2.0 ** -15: 0x7E, 2.0 ** -16: 0x07,
             0.0: 0x00, 1.5 * 2 ** 15: 0x6F, 1.25 * 2 ** 15: 0x6F, 40959.0: 0x6E, -1e-9: 0x00,
             2.0 ** -23: 0x01, -(2.0 ** -23): 0x81, 1.5 * 2 ** -16: 0x7E, 1.4999 * 2 ** -16: 0x07,
             float("inf"): 0x6F, float("-inf"): 0xEF, 1e30: 0x6F, -1e30: 0xEF}
    x = np.array(list(cases), dtype=np.float32)
    got = O.encode(x, O.F32, rnd=O.TA)
    assert [int(g) for g in got] == list(cases.values())
    assert int(O.encode(np.array([-0.0], np.float32), O.F32)[0]) == 0x00
    assert int(O.encode(np.array([np.nan], np.float32), O.F32)[0]) == 0x80
    # options (Section 3): saturation to boundary on overflow, NaN to zero
    sat = O.encode(np.array([1e30, -np.inf, 40960.0, np.nan], np.float32), O.F32, flags=O.SATURATE)
    assert [int(v) for v in sat] == [0x6E, 0xEE, 0x6E, 0x80]
    nz = O.encode(np.array([np.nan, np.inf], np.float32), O.F32, flags=O.NAN_TO_ZERO)
    assert [int(v) for v in nz] == [0x00, 0x6F]


@pytest.mark.parametrize("dtype", DT16)
def test_ta_half_ulp_bound_nearest_and_ties(dtype):
    # Section 3.1: rounding half has an error of 0.5 ulp; exact ties go away from zero
    bits = W.all_u16()
    x = src_values(bits, dtype)
    codes = O.encode(bits, dtype, rnd=O.TA)
    mags = pos_magnitudes()
    for i in np.nonzero(np.isfinite(x))[0][::7]:
        a = Fraction(abs(x[i]))
        got = Fraction(abs(O.parse(int(codes[i]))["value"]))
        if a >= 49152:
            assert got == 49152
            continue
        lo, hi = neighbours(a, mags)
        assert got in (lo, hi)
        assert abs(got - a) <= (hi - lo) / 2            # 0.5 ulp
        if a - lo == hi - a:
            assert got == hi                            # tie away from zero
        if got != 0:
            assert (int(codes[i]) >> 7) == int(np.signbit(x[i]))
    assert np.all(codes[np.isnan(x)] == 0x80)


@pytest.mark.parametrize("mode", MODES)
def test_idempotent_on_representable_values(mode):
    codes = np.array(finite_codes() + [0x00, 0x6F, 0xEF, 0x80], dtype=np.uint8)
    for dtype in (O.F32, O.BF16, O.F16):
        src = O.decode(codes, dtype)
        for seed in (0, 1, 99):
            back = O.encode(src, dtype, rnd=mode, seed=seed)
            assert np.array_equal(back, codes), (mode, dtype)


@pytest.mark.parametrize("mode", [O.TA, O.TE])
def test_monotone_and_odd(mode):
    bits = W.all_u16()
    tab = np.array([O.value(c) for c in range(256)])
    tab = np.clip(np.nan_to_num(tab, nan=0.0, posinf=1e9, neginf=-1e9), -1e9, 1e9)
    for dtype in DT16:
        x = src_values(bits, dtype)
        v = tab[O.encode(bits, dtype, rnd=mode)]
        ok = np.isfinite(x)
        order = np.argsort(x[ok], kind="stable")
        assert np.all(np.diff(v[ok][order]) >= 0)       # x <= x' => enc(x) <= enc(x')
        pos = bits[(bits & 0x8000) == 0]
        vp = tab[O.encode(pos, dtype, rnd=mode)]
        vn = tab[O.encode(pos | 0x8000, dtype, rnd=mode)]
        fin = np.isfinite(src_values(pos, dtype))
        assert np.array_equal(vn[fin], -vp[fin])        # odd symmetry (zero has a single pattern)


def test_te_tie_probability_and_te_vs_ta():
    # Section 3.1: with a 3-bit mantissa kept, the TE special case has probability 2^-20 for FP32 sources.
    first = int(np.float32(1.0).view(np.uint32))
    n = 1 << 23                                         # the whole binade [1, 2)
    ta = O.encode_f32_range(first, n, rnd=O.TA, quick=True)
    te = O.encode_f32_range(first, n, rnd=O.TE, quick=True)
    diff = np.nonzero(ta != te)[0]
    m = np.arange(n, dtype=np.int64)
    ties = np.nonzero((m & ((1 << 20) - 1)) == (1 << 19))[0]      # discarded bits = 100...0
    assert len(ties) / n == 2.0 ** -20
    even_kept = [t for t in ties if ((t >> 20) & 1) == 0]         # kept LSB already even -> TE stays
    assert list(diff) == even_kept
    # the brute-force scan agrees with the neighbour-pair variant on the ties and around them
    idx = np.unique(np.concatenate([ties, ties - 1, ties + 1, np.arange(0, n, 4099)])) % n
    x = (np.uint32(first) + idx.astype(np.uint32)).view(np.float32)
    for mode in (O.TA, O.TE):
        assert np.array_equal(O.encode(x, O.F32, rnd=mode, quick=False),
                              O.encode(x, O.F32, rnd=mode, quick=True))


def test_te_special_binades():
    # READING pinned: kept-significand parity counts the implicit one; below 2^-22 it is 0
    x = np.array([1.5 * 2 ** -20, 2.0 ** -23, 1.25 * 2 ** 15, 18.0, 22.0], dtype=np.float32)
    assert [O.value(c) for c in O.encode(x, O.F32, rnd=O.TE)] == [2.0 ** -19, 0.0, 2.0 ** 15, 16.0, 24.0]


def test_scan_equals_pair_variant_exhaustive_16bit():
    bits = W.all_u16()
    for dtype in DT16:
        for mode in (O.TA, O.TE):
            for se in (0, 3, -9):
                assert np.array_equal(O.encode(bits, dtype, scale_exp=se, rnd=mode, quick=False),
                                      O.encode(bits, dtype, scale_exp=se, rnd=mode, quick=True))


@pytest.mark.parametrize("dtype", DT16)
def test_sr2_thresholds_and_error_bound(dtype):
    # Section 3.2: SR2 has only the thresholds 0.25 and 0.75 and a rounding error of at most 0.75 ulp
    bits = W.all_u16()
    x = src_values(bits, dtype)
    codes = O.encode(bits, dtype, rnd=O.SSR)
    mags = pos_magnitudes()
    worst = Fraction(0)
    for i in np.nonzero(np.isfinite(x))[0][::5]:
        a = Fraction(abs(x[i]))
        if a >= 49152:
            continue
        lo, hi = neighbours(a, mags)
        F = (a - lo) / (hi - lo)
        got = Fraction(abs(O.parse(int(codes[i]))["value"]))
        thr = Fraction(3, 4) if (int(bits[i]) & 1) else Fraction(1, 4)
        assert got == (hi if F >= thr else lo), (hex(int(bits[i])), float(F))
        worst = max(worst, abs(got - a) / (hi - lo))
    assert worst == Fraction(3, 4)


def test_sr14_error_bound_and_unbiased():
    # Section 3.2: SR14 keeps the 1 ulp error of standard SR; the low source bits act as the threshold
    x = W.loguniform_f32(200000, seed=11, lo_exp=-24, hi_exp=16)
    codes = O.encode(x, O.F32, rnd=O.SSR)
    vals = np.array([O.parse(c)["value"] for c in range(256)])
    got = np.abs(vals[codes])
    cand = np.array([0.0] + [float(v) for v in pos_magnitudes()] + [49152.0])
    a = np.abs(x.astype(np.float64))
    j = np.searchsorted(cand, a, side="right") - 1
    lo, hi = cand[j], cand[np.minimum(j + 1, len(cand) - 1)]
    inr = a < 49152
    assert np.all((got[inr] == lo[inr]) | (got[inr] == hi[inr]))      # error below 1 ulp
    F = (a[inr] - lo[inr]) / (hi[inr] - lo[inr])
    up = got[inr] == hi[inr]
    T = (x.view(np.uint32)[inr] & 0x3FFF).astype(np.float64)          # 14 LSBs of the source
    F14 = np.floor(F * 16384.0)                                       # 14 MSBs of the discarded bits
    assert np.array_equal(up, (F14 != 0) & (F14 >= T))
    err = (got[inr] - a[inr]) / (hi[inr] - lo[inr])                   # mean invariance (K + F identity)
    assert abs(err.mean()) < 4 * 0.5 / np.sqrt(err.size)


def test_sr14_hand_worked_bit_level_vectors():
    # Section 3.2, SR14: one FP32 pattern per mantissa width 3 / 2 / 1 / 0 and below 2^-22, bits written out and the
    # expected neighbour derived by hand in tests/golden/sr14_hand_vectors.txt.  Each vector is chosen so that a
    # fraction taken from the wrong end of the discarded field, a width taken from the unscaled binade, a strict
    # comparison or plain nearest rounding gives a different byte.
    rows = []
    for line in open(os.path.join(GOLDEN, "sr14_hand_vectors.txt")):
        line = line.split("#")[0].split()
        if line:
            rows.append((int(line[0], 16), int(line[1]), int(line[2], 16)))
    assert len(rows) >= 11
    for bits, se, want in rows:
        src = np.array([bits], dtype=np.uint32)
        for quick in (False, True):
            assert int(O.encode(src, O.F32, se, O.SSR, quick=quick)[0]) == want, hex(bits)
        # Eq. 3: the hybrid mode is the simplified SR from |E| = 4 on
        E = int(np.floor(np.log2(abs(float(src.view(np.float32)[0]) * 2.0 ** se))))
        if abs(E) >= 4:
            assert int(O.encode(src, O.F32, se, O.HR)[0]) == want, hex(bits)
    # the vectors do tell the alternatives apart: round half away differs on most of them
    ta = [int(O.encode(np.array([b], dtype=np.uint32), O.F32, se, O.TA)[0]) for b, se, _ in rows]
    assert sum(t != w for t, (_, _, w) in zip(ta, rows)) >= 7


def test_index_addressed_entries_follow_the_flat_index():
    # standard SR draws word (i mod 4) of the Philox block i / 4 (pinned by the known-answer test above): an element
    # handed over together with its flat position gets the same code as inside the whole tensor, also far beyond 2^32
    x = W.loguniform_f32(4096, seed=21, lo_exp=-24, hi_exp=16)
    full = O.encode(x, O.F32, rnd=O.SR, seed=9)
    pick = np.random.default_rng(1).permutation(4096)[:500]
    assert np.array_equal(O.encode_at(x[pick], O.F32, pick, rnd=O.SR, seed=9), full[pick])
    fq = O.fake_quant(x, O.F32, 3, O.SR, seed=9)
    assert np.array_equal(O.fake_quant_at(x[pick], O.F32, pick, 3, O.SR, seed=9), fq[pick])
    # T = top 24 bits of the word of that index; with F just below / above T / 2^24 the neighbour flips
    base = np.uint64(1) << np.uint64(40)
    for k in range(64):
        i = int(base) + 977 * k
        T = O.sr_word(9, i) >> 8
        if T == 0:
            continue
        # value 1 + (j / 2^24) / 8 in the binade of 1.0 (ulp 1/8): F * 2^24 = j exactly for j a multiple of 2^4
        for j, up in ((T - 16) & ~15, False), ((T + 15) & ~15, True):
            if 0 < j < (1 << 24):
                v = np.array([1.0 + j / 2.0 ** 27], dtype=np.float32)
                assert float(v[0]) == 1.0 + j / 2.0 ** 27
                got = int(O.encode_at(v, O.F32, [i], rnd=O.SR, seed=9)[0])
                assert got == (0x09 if up else 0x08), (i, j, T)


@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_sr_expectation(dtype):
    # Section 3.2: E[SR] = (K+1) F + K (1-F) = K + F
    n = 1 << 16
    if dtype == O.F32:
        src = np.full(n, 1.03, dtype=np.float32)
        a = float(np.float32(1.03))
    else:
        src = W.f32_to_bf16_bits(np.full(n, 4.65625, dtype=np.float32))   # binade 2^2, spacing 0.5
        a = float(W.bf16_bits_to_f32(src[:1])[0])
    lo, hi = neighbours(Fraction(a), pos_magnitudes())
    F = float((Fraction(a) - lo) / (hi - lo))
    for seed in (1, 2):
        codes = O.encode(src, dtype, rnd=O.SR, seed=seed)
        v = np.array([O.value(c) for c in range(256)])[codes]
        assert set(np.unique(v)) <= {float(lo), float(hi)}
        p = np.mean(v == float(hi))
        assert abs(p - F) < 5 * np.sqrt(F * (1 - F) / n)
    Nbits = 24 if dtype == O.F32 else 16                # threshold definition: N-bit word, F_N >= T_N
    codes = O.encode(src[:512], dtype, rnd=O.SR, seed=5)
    FN = int(np.floor(F * 2 ** Nbits))
    for i in range(512):
        T = O.sr_word(5, i) >> (32 - Nbits)
        assert (O.value(codes[i]) == float(hi)) == (FN != 0 and FN >= T)


@pytest.mark.parametrize("dtype", DT16)
def test_hr_switch(dtype):
    # Eq. 3: TA for |E| < 4, simplified SR for |E| >= 4
    bits = W.all_u16()
    x = src_values(bits, dtype)
    for se in (0, 2):
        hr = O.encode(bits, dtype, scale_exp=se, rnd=O.HR)
        ta = O.encode(bits, dtype, scale_exp=se, rnd=O.TA)
        ssr = O.encode(bits, dtype, scale_exp=se, rnd=O.SSR)
        fin = np.isfinite(x) & (x != 0)
        E = np.floor(np.log2(np.abs(x[fin]))) + se
        small = np.abs(E) < 4
        assert np.array_equal(hr[fin][small], ta[fin][small])
        assert np.array_equal(hr[fin][~small], ssr[fin][~small])
        assert np.array_equal(hr[~fin], ta[~fin])
        assert np.any(ta[fin][~small] != ssr[fin][~small])


def test_scaling_is_exact_exponent_shift():
    # Section 4.2: power-of-two scale factors only add to the exponent
    x = W.normal_f32(5000, seed=3)
    for mode in (O.TA, O.TE, O.SSR):
        for se in (-7, 5):
            scaled = np.ldexp(x, se).astype(np.float32)
            a = O.encode(x, O.F32, scale_exp=se, rnd=mode)
            b = O.encode(scaled, O.F32, scale_exp=0, rnd=mode)   # low mantissa bits (thresholds) unchanged
            assert np.array_equal(a, b)


def test_flags_all_modes():
    x = np.array([np.nan, np.inf, -np.inf, 1e9, -1e9, 49152.0, 3.0], dtype=np.float32)
    for mode in MODES:
        c = O.encode(x, O.F32, rnd=mode, seed=3)
        assert [int(v) for v in c[:6]] == [0x80, 0x6F, 0xEF, 0x6F, 0xEF, 0x6F]
        c = O.encode(x, O.F32, rnd=mode, seed=3, flags=O.SATURATE | O.NAN_TO_ZERO)
        assert [int(v) for v in c[:6]] == [0x00, 0x6E, 0xEE, 0x6E, 0xEE, 0x6E]
        assert O.value(c[6]) == 3.0


# ----------------------------------------------------------------------------- amax / fake-quant / gemm
def test_amax_scale_closed_form():
    x = W.normal_f32(10000, seed=5)
    x[17] = np.inf
    x[18] = np.nan
    fin = x[np.isfinite(x)]
    amax, se = O.amax_scale(x, O.F32, target_exp=14)
    assert amax == float(np.max(np.abs(fin)))
    assert 2.0 ** 14 <= amax * 2.0 ** se < 2.0 ** 15
    codes = O.encode(fin, O.F32, scale_exp=se)
    assert not np.any((codes & 0x7F) == 0x6F)                       # finite input never overflows
    assert O.amax_scale(np.zeros(8, np.float32), O.F32) == (0.0, 0)
    assert O.amax_scale(np.array([2.0 ** -140], np.float32), O.F32, 14)[1] == 126
    assert O.amax_scale(np.array([3e38], np.float32), O.F32, -20)[1] == -126
    b = W.normal_bf16(4096, seed=6, std=0.02)
    amax, se = O.amax_scale(b, O.BF16, target_exp=3)
    assert amax == float(np.max(np.abs(W.bf16_bits_to_f32(b))))
    assert 8.0 <= amax * 2.0 ** se < 16.0


@pytest.mark.parametrize("dtype", [O.F32, O.BF16, O.F16])
def test_fake_quant_composition_and_idempotence(dtype):
    if dtype == O.F32:
        src = W.normal_f32(20000, seed=8)
    elif dtype == O.BF16:
        src = W.normal_bf16(20000, seed=8)
    else:
        src = W.normal_f32(20000, seed=8).astype(np.float16).view(np.uint16)
    for mode in (O.TA, O.HR):
        for se in (0, 6, -3):
            fq = O.fake_quant(src, dtype, scale_exp=se, rnd=mode)
            codes = O.encode(src, dtype, scale_exp=se, rnd=mode)
            assert np.array_equal(fq, O.decode(codes, dtype, scale_exp=se))
            if mode == O.TA:
                fq_in = fq.view(np.float32) if dtype == O.F32 else fq
                assert np.array_equal(O.fake_quant(fq_in, dtype, scale_exp=se, rnd=mode), fq)


def test_gemm_oracle_against_numpy():
    M, N, K = 13, 9, 37                                 # non-square: a transposed operand cannot pass
    Aq = W.random_codes((M, K), seed=1)
    Wq = W.random_codes((K, N), seed=2)
    tab = np.array([O.value(c) for c in range(256)])
    a, w = tab[Aq], tab[Wq]
    cs, s = O.gemm_full(Aq, Wq, False, 3, -2)
    assert np.allclose(cs, (a @ w) * 2.0 ** -1, rtol=1e-12, atol=0)
    assert np.allclose(s, (np.abs(a) @ np.abs(w)) * 2.0 ** -1, rtol=1e-12)
    cs2, _ = O.gemm_full(Aq, np.ascontiguousarray(Wq.T), True, 3, -2)
    assert np.array_equal(cs, cs2)
    rows = np.array([0, 12, 5]); cols = np.array([8, 0, 3])
    ce, se_ = O.gemm_entries(Aq, Wq, False, 3, -2, rows, cols)
    assert np.array_equal(ce, cs[rows, cols]) and np.array_equal(se_, s[rows, cols])
    # small-integer operands: exact equality with integer arithmetic
    ints = np.array([0x00, 0x08, 0x10, 0x14, 0x20, 0x88, 0x90], dtype=np.uint8)    # 0, 1, 2, 3, 4, -1, -2
    rng = np.random.default_rng(3)
    Ai = ints[rng.integers(0, len(ints), (M, K))]
    Wi = ints[rng.integers(0, len(ints), (K, N))]
    ci, _ = O.gemm_full(Ai, Wi, False, 0, 0)
    assert np.array_equal(ci, (tab[Ai].astype(np.int64) @ tab[Wi].astype(np.int64)).astype(np.float64))


def test_pts_search_against_definition_and_scale_shift_property():
    # Algorithm 1: the error table recomputed from the pinned pieces (cast, decode) with numpy's matmul, and two
    # properties of power-of-two scaling: a tensor pre-multiplied by 2^s shifts the table by s along its axis, and
    # an operand that is exactly representable at every scale contributes no error
    M, N, K = 24, 20, 48
    a = W.normal_bf16((M, K), seed=41)
    w = W.normal_bf16((K, N), seed=42, std=0.05)
    af, wf = W.bf16_bits_to_f32(a).astype(np.float64), W.bf16_bits_to_f32(w).astype(np.float64)
    Oref = (af @ wf).astype(np.float32)
    err, best = O.pts_search(a, w, O.BF16, False, Oref, -4, 5)
    tab = np.array([O.value(c) for c in range(256)])
    for ea, ew in [(-4, -4), (0, 3), (5, 5), (2, -1)]:
        aq, wq = tab[O.encode(a, O.BF16, ea)], tab[O.encode(w, O.BF16, ew)]
        want = np.mean(((aq @ wq) * 2.0 ** -(ea + ew) - Oref.astype(np.float64)) ** 2)
        assert np.isclose(err[ea + 4, ew + 4], want, rtol=1e-12)
    assert err[best[0] + 4, best[1] + 4] == err.min()
    a2 = W.f32_to_bf16_bits(W.bf16_bits_to_f32(a) * np.float32(4.0))           # A * 2^2: exact in BF16
    O2 = (af * 4.0 @ wf).astype(np.float32)
    err2, _ = O.pts_search(a2, w, O.BF16, False, O2, -4, 5)
    assert np.allclose(err2[:8, :], 16.0 * err[2:, :], rtol=1e-6)              # Ea' = Ea - 2, errors scale by 4^2
    ones = np.full((M, K), 0x3F80, dtype=np.uint16)                            # all-ones A: exact at every Ea
    O3 = (np.ones((M, K)) @ wf).astype(np.float32)
    err3, _ = O.pts_search(ones, w, O.BF16, False, O3, -4, 5)
    assert np.allclose(err3, err3[0:1, :], rtol=1e-9)                          # no dependence on Ea
    errq, bestq = O.pts_search(a, w, O.BF16, False, Oref, -4, 5, quick=True)
    assert np.allclose(errq, err, rtol=1e-12) and bestq == best      # (the parallel sum order is not fixed)
    errt, _ = O.pts_search(a, np.ascontiguousarray(w.T), O.BF16, True, Oref, -4, 5)
    assert np.allclose(errt, err, rtol=1e-12)


def test_significand_bits_over_exponent_profile():
    """The content of the paper's Fig. 1 (significand bits as a function of the exponent), recomputed from the decoded
    values alone: in every binade the positive finite values are 2^E * (1 + j / 2^w), j = 0 .. 2^w - 1, which gives the
    mantissa width w of that binade; the profile must be the tapered, symmetric one of Table 3 with the denormal tail."""
    import math
    vals = sorted({O.value(c) for c in range(128) if O.parse(c)["kind"] == 1})
    by_exp = {}
    for v in vals:
        by_exp.setdefault(math.floor(math.log2(v)), []).append(v)
    assert sorted(by_exp) == list(range(-22, 16))                          # 38 binades, none missing
    profile = {}
    for E, vs in by_exp.items():
        w = round(math.log2(len(vs))) if E != 15 else 1                    # the top binade loses its second value to Inf
        assert len(vs) == (2 ** w if E != 15 else 1)
        assert vs == [2.0 ** E * (1 + j / 2 ** w) for j in range(len(vs))]  # equally spaced: Eq. 1 with a w-bit mantissa
        profile[E] = w
    expect = {E: (0 if E <= -16 else 3 if abs(E) <= 3 else 2 if abs(E) <= 7 else 1) for E in range(-22, 16)}
    assert profile == expect
    print("significand bits (1 + mantissa) by exponent:", {E: 1 + w for E, w in profile.items()})
