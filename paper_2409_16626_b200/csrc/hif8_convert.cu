// HiF8 streaming conversion kernels for sm_100a: encode, decode, amax, fake-quant.
//
// Format: "Ascend HiFloat8 Format for Deep Learning" (arXiv 2409.16626), Section 2.1 (Tables 1-3, Eq. 1-2);
// rounding: Section 3 (TA / TE, standard and simplified stochastic rounding, Eq. 3 hybrid); scaling:
// Section 4.2 / 5.1 (power-of-two per-tensor scale, amax).
//
// Design notes
//  * Every element is first scaled with one FP32 multiply by 2^scale_exp.  The product is exact whenever it
//    matters (a normal result keeps all 24 significand bits; results below 2^-126 are far below the
//    smallest HiF8 value 2^-22), FP32 subnormal sources are normalised by the hardware, +-Inf stays +-Inf and
//    every NaN becomes one canonical pattern.
//  * Round-half-away (TA) of the scaled binary32 pattern depends only on its sign, exponent and top four
//    mantissa bits (the widest HiF8 mantissa is 3 bits plus the rounding bit), so the whole conversion is one
//    lookup in an 8 KiB table indexed by the top 13 bits; the table is built at compile time from the field
//    definitions and staged in shared memory.
//  * The other rounding methods add a method-specific increment below the kept bits (so that the carry does
//    the rounding, including across binade and mantissa-width boundaries), clear the discarded bits and use the
//    same table to pack the fields.
//  * Memory access: one 16-byte load per thread and instruction, consecutive lanes on consecutive 16-byte
//    groups, four independent groups in flight per thread; one block per 16 KiB of input so that the hardware
//    block scheduler balances the SMs.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <type_traits>

#include "hif8.h"
#include "hif8_device.cuh"
#include "hif8_internal.cuh"

namespace hif8 {

std::atomic<uint64_t> g_launches{0};

namespace {

// One group of kUnroll vectors per thread starting at vector index `base`.  FULL: the whole group lies inside the
// tensor, so no bounds are checked.
// PATTERN (FP32 only): the source is not read; element i is the FP32 value with encoding p.pattern_first + i.
template <int SRC, int MODE, bool FQ, bool AMAX, bool FULL, bool PATTERN = false>
__device__ __forceinline__ void convert_group(const ConvParams& p, const SmemTables& sm, unsigned long long base, unsigned long long n_vec,
                                              float scale, float d1, float d2, uint32_t k0, uint32_t k1, float& amax)
{
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    const uint4* src = reinterpret_cast<const uint4*>(p.src);
    uint4 v[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; j++) {
        unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
        if (PATTERN) {
            const uint32_t b = p.pattern_first + (uint32_t)(u * 4u);
            v[j] = make_uint4(b, b + 1u, b + 2u, b + 3u);
        } else if (FULL || u < n_vec) v[j] = __ldcs(src + u);
        else v[j] = make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int j = 0; j < kUnroll; j++) {
        unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
        if (!FULL && u >= n_vec) continue;
        if constexpr (SRC == HIF8_BF16 && (MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR) && !FQ) {
            // two elements per word (see encode_sum16)
            const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w}, ns2 = neg_scale_bf16x2(scale);
            uint32_t y[4], c[4];
#pragma unroll
            for (int k = 0; k < 4; k++) {
                if (AMAX) {
                    amax = amax_step(amax, __uint_as_float(w[k] << 16));
                    amax = amax_step(amax, __uint_as_float(w[k] & 0xFFFF0000u));
                }
                y[k] = mul_bf16x2(w[k], ns2);
                c[k] = encode_sum16(w[k], y[k], sm.ta, sm.thr);
            }
            // gather the codes and the sign bytes of four elements; a set (inverted) sign clears bit 7
            const uint32_t c0 = __byte_perm(c[0], c[1], 0x5410), c1 = __byte_perm(c[2], c[3], 0x5410);
            const uint32_t s0 = __byte_perm(y[0], y[1], 0x7531), s1 = __byte_perm(y[2], y[3], 0x7531);
            __stcs(reinterpret_cast<uint2*>(p.dst) + u, make_uint2(c0 & (~s0 | 0x7F7F7F7Fu), c1 & (~s1 | 0x7F7F7F7Fu)));
            continue;
        }
        if constexpr (SRC == HIF8_F32 && (MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR) && !FQ) {
            // four elements: neighbour-pair words, the comparisons pick the bytes pairwise, one sign step for all four
            const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
            uint32_t y[4], ent[4], sel[4];
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const float x = __uint_as_float(w[k]);
                if (AMAX) amax = amax_step(amax, x);
                const float ys = x * -scale;
                y[k] = __float_as_uint(ys);
                sel[k] = pair32_lookup<MODE>(ys, w[k], reinterpret_cast<const uint32_t*>(sm.ta), ent[k]) ? 1u : 0u;
            }
            const uint32_t c01 = __byte_perm(ent[0], ent[1], 0x4051u + sel[0] + (sel[1] << 4));
            const uint32_t c23 = __byte_perm(ent[2], ent[3], 0x4051u + sel[2] + (sel[3] << 4));
            const uint32_t s01 = __byte_perm(y[0], y[1], 0x7373), s23 = __byte_perm(y[2], y[3], 0x7373);
            const uint32_t c = __byte_perm(c01, c23, 0x5410), s = __byte_perm(s01, s23, 0x5410);
            __stcs(reinterpret_cast<uint32_t*>(p.dst) + u, c & (~s | 0x7F7F7F7Fu));  // a set (inverted) sign clears bit 7
            continue;
        }
        if constexpr (MODE == HIF8_RND_TA && !FQ && !PATTERN) {  // (a pattern sweep has neighbouring lanes in one table word anyway)
            // the code table is read sign-free, the signs go back onto the packed words (see ta_magnitude_code)
            uint32_t c[8];
#pragma unroll
            for (int k = 0; k < PV; k++) {
                float x; uint32_t raw;
                unpack<SRC>(v[j], k, x, raw);
                if (AMAX) amax = amax_step(amax, x);
                c[k] = ta_magnitude_code(x, scale, sm.ta);
            }
            uint32_t w0 = c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24), w1 = 0;
            if (PV == 8) w1 = c[4] | (c[5] << 8) | (c[6] << 16) | (c[7] << 24);
            put_signs<SRC>(v[j], w0, w1);
            if (PV == 4) __stcs(reinterpret_cast<uint32_t*>(p.dst) + u, w0);
            else __stcs(reinterpret_cast<uint2*>(p.dst) + u, make_uint2(w0, w1));
            continue;
        }
        uint32_t codes[PV];
        uint4 r0 = make_uint4(0, 0, 0, 0), r1 = r0;
        if (MODE == HIF8_RND_SR) {
            r0 = philox4x32_10((uint32_t)(u * (PV / 4)), (uint32_t)((u * (PV / 4)) >> 32), k0, k1);
            if (PV == 8) r1 = philox4x32_10((uint32_t)(u * 2 + 1), (uint32_t)((u * 2 + 1) >> 32), k0, k1);
        }
        const uint32_t rw[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
        for (int k = 0; k < PV; k++) {
            float x; uint32_t raw;
            unpack<SRC>(v[j], k, x, raw);
            if (AMAX) amax = amax_step(amax, x);
            codes[k] = encode_one<MODE, SRC>(x, raw, scale, sm.ta, sm.thr, rw[k]);
        }
        if (!FQ) {
            uint32_t w0 = codes[0] | (codes[1] << 8) | (codes[2] << 16) | (codes[3] << 24);
            if (PV == 4) __stcs(reinterpret_cast<uint32_t*>(p.dst) + u, w0);
            else {
                uint32_t w1 = codes[4] | (codes[5] << 8) | (codes[6] << 16) | (codes[7] << 24);
                __stcs(reinterpret_cast<uint2*>(p.dst) + u, make_uint2(w0, w1));
            }
        } else {
            uint32_t o[PV];
#pragma unroll
            for (int k = 0; k < PV; k++) o[k] = to_bits<SRC>(sm.dec[codes[k]] * d1 * d2);
            uint4 out;
            if (PV == 4) out = make_uint4(o[0], o[1], o[2], o[3]);
            else out = make_uint4(o[0] | (o[1] << 16), o[2] | (o[3] << 16), o[4] | (o[5] << 16), o[6] | (o[7] << 16));
            __stcs(reinterpret_cast<uint4*>(p.dst) + u, out);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Encode / fake-quant kernel.  FQ = false: bytes out.  FQ = true: dequantized values in the source format.
// AMAX = true: also reduce amax of the source into p.amax_accum[0]; the last block publishes it.
// ------------------------------------------------------------------------------------------------
template <int SRC, int MODE, bool FQ, bool AMAX, bool PATTERN = false>
__global__ void __launch_bounds__(kThreads) convert_kernel(const ConvParams p, unsigned long long n_vec)
{
    static_assert(!PATTERN || (SRC == HIF8_F32 && !FQ && !AMAX), "generated sources are FP32 patterns, encode only");
    __shared__ SmemTables sm;
    pdl_launch_dependents();
    constexpr bool kPair16 = SRC == HIF8_BF16 && (MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR) && !FQ;
    if (kPair16) setup_sum16<MODE>(sm.ta, sm.thr, p.flags);
    else setup_tables<true, MODE != HIF8_RND_TA, FQ, MODE, SRC>(sm, p.flags);  // reads only the constant table
    pdl_wait_prior_grid();
    const int se = resolve_scale_exp(p);
    const float scale = pow2f(se);
    const int da = (-se) / 2, db = -se - da;  // descale in two exact steps (the first cannot leave the normal range)
    const float d1 = pow2f(da), d2 = pow2f(db);
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
    float amax = 0.f;

    // group g of the tensor = vectors [g, g + 1) * kThreads * kUnroll; this block takes groups blockIdx.x, + gridDim.x, ...
    // counted from the front or (p.reverse) from the back of the tensor
    constexpr unsigned long long kGroupVecs = (unsigned long long)kThreads * kUnroll;
    const unsigned long long n_groups = (n_vec + kGroupVecs - 1) / kGroupVecs;
    for (unsigned long long g = blockIdx.x; g < n_groups; g += gridDim.x) {
        const unsigned long long base = (p.reverse ? n_groups - 1 - g : g) * kGroupVecs;
        if (base + kGroupVecs <= n_vec)
            convert_group<SRC, MODE, FQ, AMAX, true, PATTERN>(p, sm, base, n_vec, scale, d1, d2, k0, k1, amax);
        else
            convert_group<SRC, MODE, FQ, AMAX, false, PATTERN>(p, sm, base, n_vec, scale, d1, d2, k0, k1, amax);
    }
    // elements not covered by whole vectors (tail, or everything when the pointers are not 16-byte aligned)
    {
        const unsigned long long first = n_vec * PV;
        const unsigned long long tid = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
        for (unsigned long long i = first + tid; i < p.n; i += (unsigned long long)gridDim.x * kThreads) {
            float x; uint32_t raw;
            if (PATTERN) { raw = p.pattern_first + (uint32_t)i; x = __uint_as_float(raw); }
            else load_scalar<SRC>(p.src, i, x, raw);
            if (AMAX) amax = amax_step(amax, x);
            uint32_t word = 0;
            if (MODE == HIF8_RND_SR) {
                uint4 r = philox4x32_10((uint32_t)(i >> 2), (uint32_t)(i >> 34), k0, k1);
                word = philox_word(r, (unsigned)i & 3u);
            }
            uint32_t c;
            if constexpr (kPair16) {
                const uint32_t y = mul_bf16x2(raw, neg_scale_bf16x2(scale));  // the element as the low half of a word
                c = encode_sum16(raw, y, sm.ta, sm.thr) & (~(y >> 8) | 0x7Fu) & 0xFFu;
            } else c = encode_one<MODE, SRC>(x, raw, scale, sm.ta, sm.thr, word);
            if (!FQ) reinterpret_cast<uint8_t*>(p.dst)[i] = (uint8_t)c;
            else {
                uint32_t o = to_bits<SRC>(sm.dec[c] * d1 * d2);
                if (SRC == HIF8_F32) reinterpret_cast<uint32_t*>(p.dst)[i] = o;
                else reinterpret_cast<unsigned short*>(p.dst)[i] = (unsigned short)o;
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (p.d_scale_exp_out) *p.d_scale_exp_out = se;
        if (p.d_scale_out) *p.d_scale_out = scale;
        if (!AMAX && p.d_amax_out && p.d_amax_bits) *p.d_amax_out = __uint_as_float(*p.d_amax_bits);
    }
    if (AMAX) {
        block_amax_commit(amax, p.amax_accum);
        if (threadIdx.x == 0) {
            __threadfence();
            uint32_t ticket = atomicAdd(p.amax_accum + 1, 1u);
            if (ticket == gridDim.x - 1) {  // last block: every partial maximum is visible
                __threadfence();
                uint32_t ab = atomicMax(p.amax_accum, 0u);
                if (p.d_amax_out) *p.d_amax_out = __uint_as_float(ab);
                if (p.scale_state) {
                    // delayed scaling: every block has read the exponent in force and finished, so the state can move on;
                    // the accumulator and the ticket are left at zero for the next measuring pass
                    scale_state_push(reinterpret_cast<ScaleState*>(p.scale_state), ab, p.target_exp);
                    p.amax_accum[0] = 0u;
                    p.amax_accum[1] = 0u;
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Fake-quant with the rounding done on the source bit pattern itself: round half away (FP32, BF16), and hybrid /
// simplified stochastic rounding (BF16).
// A power-of-two scale only moves which HiF8 binade (hence mantissa width) a source exponent falls into, so
// quantize-dequantize is "add half of the discarded field, clear it" with an increment and a mask looked up by the
// source exponent (table rebuilt per block for the scale in force).  No multiply, no code byte, no value table.
// Exponents whose result is not of that form (overflow and the binade below it, Inf / NaN, subnormal sources under
// a very large scale) are flagged in the table and take a table-free per-element routine.
// ------------------------------------------------------------------------------------------------
constexpr uint32_t kRareMask = 1u;  // never a legitimate mask: legitimate ones are 0 or end in at least four zero bits

// one element, any input: value-level rounding through the scaled binary32 value.
// MODE: round half away, round half to even, or (BF16 sources) the 2-bit simplified stochastic rounding SR2 / hybrid
// rounding of Eq. 3.
// MODE = standard stochastic rounding (BF16 sources): T16 is the 16-bit threshold of the element (Section 3.2: one is added
// to the kept bits iff the discarded fraction, taken to 16 bits, is non-zero and at least T).
template <int SRC, int MODE>
__device__ __noinline__ uint32_t fq_rare(uint32_t raw, int se, unsigned flags, uint32_t T16 = 0u)
{
    const float x = __uint_as_float(SRC == HIF8_F32 ? raw : raw << 16);
    const float y = x * pow2f(se);
    const uint32_t t = __float_as_uint(y);
    const uint32_t a = t & 0x7FFFFFFFu, sign = t & 0x80000000u;
    if (a > 0x7F800000u) return (flags & HIF8_FLAG_NAN_TO_ZERO) ? 0u : (SRC == HIF8_F32 ? 0x7FC00000u : 0x7FC0u);
    const uint32_t top = (flags & HIF8_FLAG_SATURATE) ? 0x47000000u : 0x7F800000u;  // 2^15 or Inf
    const int E = (int)(a >> 23) - 127;
    uint32_t r;
    if (MODE == HIF8_RND_TE) {
        if (a <= 0x34000000u) return 0u;                                                   // up to the tie 2^-23 (kept significand 0 is even)
        else if (E < -22) r = 0x34800000u;                                                 // (2^-23, 2^-22) -> 2^-22
        else {
            // half - 1 plus the kept LSB; where no mantissa bit is kept the bit above the field is the implicit one (odd)
            const uint32_t k = 23u - (uint32_t)mant_width(E);
            r = (a + (1u << (k - 1)) - 1u + (k == 23u ? 1u : (a >> k) & 1u)) & (0xFFFFFFFFu << k);
            if (r >= 0x47400000u) r = top;                                                 // 1.5 * 2^15 and above
        }
    } else if (MODE == HIF8_RND_TA || (MODE == HIF8_RND_HR && E > -4 && E < 4)) {
        if (a >= 0x47200000u) r = top;                                                     // >= 1.25 * 2^15
        else if (a < 0x34000000u) return 0u;                                               // < 2^-23: the single zero
        else if (E < -22) r = 0x34800000u;                                                 // [2^-23, 2^-22) -> 2^-22
        else { const uint32_t k = 23u - (uint32_t)mant_width(E); r = (a + (1u << (k - 1))) & (0xFFFFFFFFu << k); }
    } else if (MODE == HIF8_RND_SR) {
        if (a >= 0x47400000u) r = top;                                                     // >= 1.5 * 2^15
        else if (E < -22) {                                                                // F = |y| / 2^-22, F16 = floor(2^16 F)
            const uint32_t f16 = E < -38 ? 0u : (uint32_t)floorf(fabsf(y) * 274877906944.f);  // |y| * 2^38, exact: < 2^16
            if (f16 == 0u || f16 < T16) return 0u;
            r = 0x34800000u;
        } else {
            const uint32_t k = 23u - (uint32_t)mant_width(E);                              // >= 20: the low 16 bits of a are zero
            const uint32_t f16 = (a & ((1u << k) - 1u)) >> (k - 16);
            r = (a & (0xFFFFFFFFu << k)) + (((f16 != 0u && f16 >= T16) ? 1u : 0u) << k);
            if (r >= 0x47400000u) r = top;
        }
    } else {
        const uint32_t T2 = 2u * (raw & 1u) + 1u;                                          // {source LSB, fixed 1}
        if (a >= 0x47400000u) r = top;                                                     // >= 1.5 * 2^15
        else if (E < -22) {                                                                // F = |y| / 2^-22, F2 = floor(4 F)
            if ((uint32_t)floorf(fabsf(y) * 16777216.f) < T2) return 0u;
            r = 0x34800000u;
        } else {
            const uint32_t k = 23u - (uint32_t)mant_width(E);
            const uint32_t f2 = (a & ((1u << k) - 1u)) >> (k - 2);
            r = (a & (0xFFFFFFFFu << k)) + ((f2 >= T2 ? 1u : 0u) << k);
            if (r >= 0x47400000u) r = top;
        }
    }
    const int da = (-se) / 2, db = -se - da;
    return to_bits<SRC>(__uint_as_float(r | sign) * pow2f(da) * pow2f(db));
}

// MODE = round half away (FP32, BF16), or hybrid / simplified stochastic rounding (BF16 only, in packed BF16 arithmetic:
// SR2 adds 0.75 ulp - LSB * 0.5 ulp to the magnitude, i.e. thresholds 0.25 / 0.75, where round-half-away adds half)
// MODE = round half to even (BF16 only) is done in packed BF16 arithmetic instead: (x + C) - C with C = 2^(7 - width) times
// the element's own power of two and the element's sign.  The sum lies in the binade of C, whose spacing is the HiF8
// spacing of the element's binade (2^-22 over the scale below the format's range), so the hardware's round-to-nearest-even
// does the rounding, ties to the even kept significand (the implicit one counts), and x - x = +0 gives the single zero.
template <int SRC, int MODE>
__global__ void __launch_bounds__(kThreads) fq_ta_kernel(const ConvParams p, unsigned long long n_vec)
{
    static_assert(MODE == HIF8_RND_TA || SRC == HIF8_BF16, "threshold modes and round half to even are done in place for BF16 only");
    constexpr int MB = SRC == HIF8_F32 ? 23 : 7;      // mantissa bits of the source format
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    constexpr bool kThr = MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR;  // packed BF16 arithmetic with an LSB term
    __shared__ uint32_t s_inc[256];                   // BF16: mask16 | inc16 << 16 (threshold modes: mask16 | addend << 16)
    __shared__ uint32_t s_mask[(SRC == HIF8_F32 || kThr) ? 256 : 1];  // threshold modes: the LSB term's factor
    pdl_launch_dependents();
    pdl_wait_prior_grid();  // the scale may come from the previous kernel
    const int se = resolve_scale_exp(p);
    {
        const int e = threadIdx.x, E = e - 127 + se;
        uint32_t inc = 0, mask = 0, kfac = 0;
        // (subnormal sources: below 2^(se - 126); standard SR can still round up from 2^-38 on, the other modes from 2^-24)
        if (e == 255 || (e == 0 && se > (MODE == HIF8_RND_SR ? 88 : 100)) || (e > 0 && E >= 15)) mask = kRareMask;
        else if ((MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR) && e > 0 && (E == -23 || E == -24)) mask = kRareMask;  // result is 0 or 2^-22
        else if (MODE == HIF8_RND_SR && e > 0 && E <= -23 && E >= -38) mask = kRareMask;    // 0 or 2^-22, by the threshold
        else if (e == 0 || E <= -24) { inc = 0; mask = 0; }                                 // underflow to +0
        else if (E == -23) { inc = 1u << MB; mask = 0xFFFFFFFFu << MB; }                    // up to 2^-22
        else {
            const uint32_t k = (uint32_t)(MB - mant_width(E));
            inc = 1u << (k - 1);
            mask = 0xFFFFFFFFu << k;
            if (kThr) {
                // BF16 values in the source's own scale: the addend 0.75 ulp (0.5 ulp in a round-half-away binade of
                // Eq. 3: every binade with |E| < 4 under hybrid rounding) and the factor -2^(6 - width) that turns the
                // element's own LSB (2^-7 of its power of two) into LSB * 0.5 ulp
                const int w = mant_width(E), hb = e - w - 1;  // biased exponent of 0.5 ulp
                const bool sr2 = MODE == HIF8_RND_SSR || E <= -4 || E >= 4;
                if (hb < 1) mask = kRareMask;
                else { inc = ((uint32_t)hb << 7) | (sr2 ? 0x40u : 0u); kfac = sr2 ? (0x8000u | ((uint32_t)(133 - w) << 7)) : 0u; }
            }
        }
        if (MODE == HIF8_RND_TE) {
            // biased exponent of C: the element's plus 7 - width, or that of 2^(-22 - se + 7) below the format's range
            const int cb = (e == 0 || E < -22) ? 112 - se : e + 7 - mant_width(E);
            const bool rare = mask == kRareMask || cb < 1 || cb > 254;
            s_inc[e] = rare ? kRareMask : (uint32_t)cb << 23;  // C in the high half
        } else if (SRC == HIF8_F32) { s_inc[e] = inc; s_mask[e] = mask; }
        else if (MODE == HIF8_RND_SR) {
            // mask16 | (16 - discarded bits) << 16; exponents that underflow to +0 keep mask 0 and a shift of 16 (no increment)
            const uint32_t kbits = (mask == kRareMask || mask == 0u) ? 0u : (uint32_t)__popc(~mask & 0xFFFFu);
            s_inc[e] = (mask & 0xFFFFu) | ((16u - kbits) << 16);
        } else {
            s_inc[e] = (mask & 0xFFFFu) | (inc << 16);
            if (kThr) s_mask[e] = kfac;
        }
    }
    __syncthreads();

    const uint4* src = reinterpret_cast<const uint4*>(p.src);
    // one group of kUnroll vectors per thread; a group wholly inside the tensor runs without bounds checks
    auto group = [&](unsigned long long base, auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        uint4 v[kUnroll];
#pragma unroll
        for (int j = 0; j < kUnroll; j++) {
            unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
            v[j] = (FULL || u < n_vec) ? __ldcs(src + u) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < kUnroll; j++) {
            unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
            if (!FULL && u >= n_vec) continue;
            uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w}, o[4], rare = 0;
            if (SRC == HIF8_F32) {
                uint32_t m[4];
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    const uint32_t e = (w[k] >> 23) & 0xFFu;
                    m[k] = s_mask[e];
                    o[k] = (w[k] + s_inc[e]) & m[k];
                    rare |= m[k];
                }
                if (rare & kRareMask) {
#pragma unroll
                    for (int k = 0; k < 4; k++)
                        if (m[k] == kRareMask) o[k] = fq_rare<SRC, MODE>(w[k], se, p.flags);
                }
            } else if (MODE == HIF8_RND_SR) {
                // Standard SR on the source pattern: with k discarded bits and threshold T, one is added to the kept bits iff
                // the discarded field d is non-zero and d * 2^(16 - k) >= T, i.e. iff d >= max(1, ceil(T / 2^(16 - k))): add
                // (2^k - 1) - ((max(T, 1) - 1) >> (16 - k)) and let the carry out of the field do it, then clear the field.
                // Element 8 u + j takes word j mod 4 of the Philox block 2 u + j / 4.
                const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
                const uint4 q0 = philox4x32_10((uint32_t)(u * 2), (uint32_t)((u * 2) >> 32), k0, k1);
                const uint4 q1 = philox4x32_10((uint32_t)(u * 2 + 1), (uint32_t)((u * 2 + 1) >> 32), k0, k1);
                const uint32_t rw[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
                uint32_t tl[4], th[4];
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    tl[k] = s_inc[(w[k] >> 7) & 0xFFu];
                    th[k] = s_inc[(w[k] >> 23) & 0xFFu];
                    const uint32_t Tl = rw[2 * k] >> 16, Th = rw[2 * k + 1] >> 16, sl = tl[k] >> 16, sh = th[k] >> 16;  // s = 16 - k
                    // (2^k - 1) - d per half; flagged and underflowing exponents carry s = 16: no increment at all
                    const uint32_t il = (0xFFFFu >> sl) - ((Tl - (Tl != 0u)) >> sl), ih = (0xFFFFu >> sh) - ((Th - (Th != 0u)) >> sh);
                    const uint32_t mask2 = __byte_perm(tl[k], th[k], 0x5410);
                    o[k] = (w[k] + (il | (ih << 16))) & mask2;  // no carry between the halves: only finite, in-range values add
                    rare |= tl[k] | th[k];
                }
                if (rare & kRareMask) {
#pragma unroll
                    for (int k = 0; k < 4; k++) {
                        if (tl[k] & kRareMask) o[k] = (o[k] & 0xFFFF0000u) | fq_rare<SRC, MODE>(w[k] & 0xFFFFu, se, p.flags, rw[2 * k] >> 16);
                        if (th[k] & kRareMask) o[k] = (o[k] & 0x0000FFFFu) | (fq_rare<SRC, MODE>(w[k] >> 16, se, p.flags, rw[2 * k + 1] >> 16) << 16);
                    }
                }
            } else {
                uint32_t tl[4], th[4];
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    tl[k] = s_inc[(w[k] >> 7) & 0xFFu];
                    th[k] = s_inc[(w[k] >> 23) & 0xFFu];
                    if (MODE == HIF8_RND_TE) {
                        const uint32_t cs = __byte_perm(tl[k], th[k], 0x7632) | (w[k] & 0x80008000u);  // C with the element's sign
                        o[k] = fma_bf16x2(fma_bf16x2(w[k], 0x3F803F80u, cs), 0x3F803F80u, cs ^ 0x80008000u);
                        rare |= tl[k] | th[k];
                        continue;
                    }
                    const uint32_t mask2 = __byte_perm(tl[k], th[k], 0x5410);
                    const uint32_t inc2 = __byte_perm(tl[k], th[k], 0x7632);
                    if (kThr) {
                        // SR2 rounds up iff F >= T2 / 4: x + sign * (0.75 ulp - LSB * 0.5 ulp), then the discarded bits
                        // are cleared.  The addend lies on the significand's grid, so the sum is exact unless it carries
                        // into the next binade, where what is left stays below the mask's cut.
                        const uint32_t kl = s_mask[(w[k] >> 7) & 0xFFu], kh = s_mask[(w[k] >> 23) & 0xFFu];
                        const uint32_t lsbval = fma_bf16x2(w[k] & 0xFFFEFFFEu, 0xBF80BF80u, w[k]);  // x minus x without its LSB
                        const uint32_t adds = fma_bf16x2(lsbval, __byte_perm(kl, kh, 0x5410), inc2 | (w[k] & 0x80008000u));
                        o[k] = fma_bf16x2(w[k], 0x3F803F80u, adds) & mask2;
                    } else o[k] = (w[k] + inc2) & mask2;  // no carry between the halves: flagged exponents add nothing
                    rare |= tl[k] | th[k];
                }
                if (rare & kRareMask) {
#pragma unroll
                    for (int k = 0; k < 4; k++) {
                        if (tl[k] & kRareMask) o[k] = (o[k] & 0xFFFF0000u) | fq_rare<SRC, MODE>(w[k] & 0xFFFFu, se, p.flags);
                        if (th[k] & kRareMask) o[k] = (o[k] & 0x0000FFFFu) | (fq_rare<SRC, MODE>(w[k] >> 16, se, p.flags) << 16);
                    }
                }
            }
            __stcs(reinterpret_cast<uint4*>(p.dst) + u, make_uint4(o[0], o[1], o[2], o[3]));
        }
    };
    {
        constexpr unsigned long long kGroupVecs = (unsigned long long)kThreads * kUnroll;
        const unsigned long long n_groups = (n_vec + kGroupVecs - 1) / kGroupVecs;
        for (unsigned long long g = blockIdx.x; g < n_groups; g += gridDim.x) {  // from the back of the tensor with p.reverse
            const unsigned long long base = (p.reverse ? n_groups - 1 - g : g) * kGroupVecs;
            if (base + kGroupVecs <= n_vec) group(base, std::true_type{});
            else group(base, std::false_type{});
        }
    }
    {   // tail / unaligned elements
        const unsigned long long tid = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
        for (unsigned long long i = n_vec * PV + tid; i < p.n; i += (unsigned long long)gridDim.x * kThreads) {
            if (SRC == HIF8_F32) {
                const uint32_t raw = reinterpret_cast<const uint32_t*>(p.src)[i];
                reinterpret_cast<uint32_t*>(p.dst)[i] = fq_rare<SRC, MODE>(raw, se, p.flags);
            } else {
                const uint32_t raw = reinterpret_cast<const unsigned short*>(p.src)[i];
                uint32_t T16 = 0u;
                if (MODE == HIF8_RND_SR) {
                    const uint4 q = philox4x32_10((uint32_t)(i >> 2), (uint32_t)(i >> 34), (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
                    T16 = philox_word(q, (unsigned)i & 3u) >> 16;
                }
                reinterpret_cast<unsigned short*>(p.dst)[i] = (unsigned short)fq_rare<SRC, MODE>(raw, se, p.flags, T16);
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (p.d_scale_exp_out) *p.d_scale_exp_out = se;
        if (p.d_scale_out) *p.d_scale_out = pow2f(se);
        if (p.d_amax_out && p.d_amax_bits) *p.d_amax_out = __uint_as_float(*p.d_amax_bits);
    }
}

// Clears the amax accumulator and its ticket.  A kernel rather than a memset so that the amax kernel that follows can be
// launched programmatically: its blocks become resident while this one drains and wait at their first global access.
__global__ void clear_accum_kernel(uint32_t* accum)
{
    pdl_launch_dependents();
    pdl_wait_prior_grid();
    if (threadIdx.x < 2) accum[threadIdx.x] = 0u;
}

// amax only (first pass of just-in-time scaling).  A read-only pass: eight 16-byte loads in flight per thread (32 KiB per
// block) measured 2 us faster on a 64 MiB tensor than the four of the converting kernels.
constexpr int kUnrollAmax = 8;
template <int SRC>
__global__ void __launch_bounds__(kThreads) amax_kernel(const void* __restrict__ srcv, unsigned long long n,
                                                        unsigned long long n_vec, uint32_t* accum, float* d_amax_out)
{
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    const uint4* src = reinterpret_cast<const uint4*>(srcv);
    float amax = 0.f;
    pdl_launch_dependents();
    pdl_wait_prior_grid();
    const unsigned long long stride = (unsigned long long)gridDim.x * kThreads * kUnrollAmax;
    for (unsigned long long base = (unsigned long long)blockIdx.x * kThreads * kUnrollAmax; base < n_vec; base += stride) {
        uint4 v[kUnrollAmax];
#pragma unroll
        for (int j = 0; j < kUnrollAmax; j++) {
            unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
            v[j] = (u < n_vec) ? __ldg(src + u) : make_uint4(0, 0, 0, 0);  // default policy: keep lines for the second pass
        }
#pragma unroll
        for (int j = 0; j < kUnrollAmax; j++) {
#pragma unroll
            for (int k = 0; k < PV; k++) {
                float x; uint32_t raw;
                unpack<SRC>(v[j], k, x, raw);
                amax = amax_step(amax, x);
            }
        }
    }
    const unsigned long long tid = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
    for (unsigned long long i = n_vec * PV + tid; i < n; i += (unsigned long long)gridDim.x * kThreads) {
        float x; uint32_t raw;
        load_scalar<SRC>(srcv, i, x, raw);
        amax = amax_step(amax, x);
    }
    block_amax_commit(amax, accum);
    if (d_amax_out && threadIdx.x == 0) {  // stand-alone amax: the last block to finish publishes the result
        __threadfence();
        if (atomicAdd(accum + 1, 1u) == gridDim.x - 1) {
            __threadfence();
            *d_amax_out = __uint_as_float(atomicMax(accum, 0u));
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Decode kernel: bytes -> DT, times 2^-scale_exp
// ------------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(kThreads) decode_kernel(const uint8_t* __restrict__ src, void* __restrict__ dst,
                                                          unsigned long long n, unsigned long long n_vec, int se)
{
    // Output encodings of all 256 bytes for this call: value * 2^-scale_exp in two exact power-of-two steps (the first
    // cannot leave the normal range, so only the second may round -- to nearest even), then the destination format.
    __shared__ uint32_t s_out[256];
    pdl_launch_dependents();
    {
        const int da = (-se) / 2, db = -se - da;
        s_out[threadIdx.x] = to_bits<DT>(__uint_as_float(decode_bits_f32(threadIdx.x)) * pow2f(da) * pow2f(db));
    }
    __syncthreads();
    pdl_wait_prior_grid();
    constexpr int PV = SrcTraits<DT>::kPerVec;  // codes per 16-byte store
    const unsigned long long stride = (unsigned long long)gridDim.x * kThreads * kUnroll;
    // one group of kUnroll vectors per thread; a group wholly inside the tensor runs without bounds checks
    auto group = [&](unsigned long long base, auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        uint2 v[kUnroll];
#pragma unroll
        for (int j = 0; j < kUnroll; j++) {
            unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
            v[j] = make_uint2(0, 0);
            if (FULL || u < n_vec) {
                if (PV == 4) v[j].x = __ldcs(reinterpret_cast<const uint32_t*>(src) + u);
                else v[j] = __ldcs(reinterpret_cast<const uint2*>(src) + u);
            }
        }
#pragma unroll
        for (int j = 0; j < kUnroll; j++) {
            unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
            if (!FULL && u >= n_vec) continue;
            uint32_t o[PV];
#pragma unroll
            for (int k = 0; k < PV; k++) o[k] = s_out[((k < 4 ? v[j].x : v[j].y) >> (8 * (k & 3))) & 0xFFu];
            uint4 out;
            if (PV == 4) out = make_uint4(o[0], o[1], o[2], o[3]);
            else out = make_uint4(o[0] | (o[1] << 16), o[2] | (o[3] << 16), o[4] | (o[5] << 16), o[6] | (o[7] << 16));
            __stcs(reinterpret_cast<uint4*>(dst) + u, out);
        }
    };
    for (unsigned long long base = (unsigned long long)blockIdx.x * kThreads * kUnroll; base < n_vec; base += stride) {
        if (base + (unsigned long long)kThreads * kUnroll <= n_vec) group(base, std::true_type{});
        else group(base, std::false_type{});
    }
    const unsigned long long tid = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
    for (unsigned long long i = n_vec * PV + tid; i < n; i += (unsigned long long)gridDim.x * kThreads) {
        const uint32_t o = s_out[src[i]];
        if (DT == HIF8_F32) reinterpret_cast<uint32_t*>(dst)[i] = o;
        else reinterpret_cast<unsigned short*>(dst)[i] = (unsigned short)o;
    }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
int g_sm_count[64];
int g_cc[64];

int device_info(int* sms)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HIF8_ERR_CUDA;
    if (g_sm_count[dev] == 0) {
        int n = 0, major = 0, minor = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return HIF8_ERR_CUDA;
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev);
        g_cc[dev] = major * 10 + minor;
        g_sm_count[dev] = n;
    }
    if (g_cc[dev] != 100) return HIF8_ERR_CUDA;
    *sms = g_sm_count[dev];
    return HIF8_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr int kGroupsConvert = 4;  // encode / fake-quant kernels: groups per block on large tensors

unsigned grid_for(unsigned long long n_vec, unsigned long long n, int sms, int unroll = kUnroll, int max_groups = 1)
{
    // Many more blocks than the SMs can hold, no persistent loop: blocks are handed to SMs as they free up, which
    // balances the load between SMs near to and far from a memory partition (measured 10-20 % faster than a static
    // grid-stride split).  The scalar fallback (unaligned pointers) keeps a bounded grid-stride grid.
    unsigned long long per_block = (unsigned long long)kThreads * unroll;
    unsigned long long need;
    if (n_vec) {
        need = (n_vec + per_block - 1) / per_block;
        // Large tensors: up to max_groups groups per block (grid-stride), as long as at least one full wave of resident
        // blocks remains for the scheduler to balance.  The per-block prologue (table set-up, scale) is then paid
        // once per 64 KiB instead of once per 16 KiB, which the arithmetic-bound rounding modes feel most.
        const unsigned long long wave = (unsigned long long)sms * kBlocksPerSM;
        const unsigned long long groups = need / wave < (unsigned long long)max_groups ? need / wave : (unsigned long long)max_groups;
        if (groups > 1) need = (need + groups - 1) / groups;
    } else {
        need = (n + kThreads - 1) / kThreads;
        unsigned long long cap = (unsigned long long)sms * kBlocksPerSM * 4;
        if (need > cap) need = cap;
    }
    if (need == 0) need = 1;
    if (need > 0x7FFFFFFFull) need = 0x7FFFFFFFull;
    return (unsigned)need;
}

template <int SRC, int MODE, bool FQ, bool AMAX>
int launch_convert(const ConvParams& p, bool vec_ok, int sms, cudaStream_t st)
{
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    unsigned long long n_vec = vec_ok ? p.n / PV : 0;
    unsigned grid = grid_for(n_vec, p.n, sms, kUnroll, kGroupsConvert);
    launch_pdl(convert_kernel<SRC, MODE, FQ, AMAX>, grid, st, p, n_vec);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

template <int SRC, bool FQ, bool AMAX>
int dispatch_mode(int rnd, const ConvParams& p, bool vec_ok, int sms, cudaStream_t st)
{
    switch (rnd) {
        case HIF8_RND_TA: return launch_convert<SRC, HIF8_RND_TA, FQ, AMAX>(p, vec_ok, sms, st);
        case HIF8_RND_HR: return launch_convert<SRC, HIF8_RND_HR, FQ, AMAX>(p, vec_ok, sms, st);
        case HIF8_RND_SSR: return launch_convert<SRC, HIF8_RND_SSR, FQ, AMAX>(p, vec_ok, sms, st);
        case HIF8_RND_TE: return launch_convert<SRC, HIF8_RND_TE, FQ, AMAX>(p, vec_ok, sms, st);
        default: return launch_convert<SRC, HIF8_RND_SR, FQ, AMAX>(p, vec_ok, sms, st);
    }
}

template <bool FQ, bool AMAX>
int dispatch_convert(int dtype, int rnd, const ConvParams& p, bool vec_ok, int sms, cudaStream_t st)
{
    switch (dtype) {
        case HIF8_F32: return dispatch_mode<HIF8_F32, FQ, AMAX>(rnd, p, vec_ok, sms, st);
        case HIF8_BF16: return dispatch_mode<HIF8_BF16, FQ, AMAX>(rnd, p, vec_ok, sms, st);
        default: return dispatch_mode<HIF8_F16, FQ, AMAX>(rnd, p, vec_ok, sms, st);
    }
}

int launch_fq_ta(int dtype, int rnd, const ConvParams& p, bool vec_ok, int sms, cudaStream_t st)
{
    const unsigned long long pv = dtype == HIF8_F32 ? 4 : 8;
    const unsigned long long n_vec = vec_ok ? p.n / pv : 0;
    // round half away is bound by memory here and runs best with one group per block (42.3 against 43.6 us per 2^26
    // BF16 elements); the threshold modes carry more arithmetic per element and gain from sharing the prologue
    const unsigned grid = grid_for(n_vec, p.n, sms, kUnroll, rnd == HIF8_RND_TA ? 1 : kGroupsConvert);
    if (dtype == HIF8_F32) launch_pdl(fq_ta_kernel<HIF8_F32, HIF8_RND_TA>, grid, st, p, n_vec);
    else if (rnd == HIF8_RND_TA) launch_pdl(fq_ta_kernel<HIF8_BF16, HIF8_RND_TA>, grid, st, p, n_vec);
    else if (rnd == HIF8_RND_HR) launch_pdl(fq_ta_kernel<HIF8_BF16, HIF8_RND_HR>, grid, st, p, n_vec);
    else if (rnd == HIF8_RND_TE) launch_pdl(fq_ta_kernel<HIF8_BF16, HIF8_RND_TE>, grid, st, p, n_vec);
    else if (rnd == HIF8_RND_SR) launch_pdl(fq_ta_kernel<HIF8_BF16, HIF8_RND_SR>, grid, st, p, n_vec);
    else launch_pdl(fq_ta_kernel<HIF8_BF16, HIF8_RND_SSR>, grid, st, p, n_vec);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

int launch_amax(const void* src, int dtype, unsigned long long n, uint32_t* accum, float* d_amax_out, int sms, cudaStream_t st)
{
    bool vec_ok = aligned16(src);
    unsigned long long pv = dtype == HIF8_F32 ? 4 : 8;
    unsigned long long n_vec = vec_ok ? n / pv : 0;
    unsigned grid = grid_for(n_vec, n, sms, kUnrollAmax);
    switch (dtype) {
        case HIF8_F32: launch_pdl(amax_kernel<HIF8_F32>, grid, st, src, n, n_vec, accum, d_amax_out); break;
        case HIF8_BF16: launch_pdl(amax_kernel<HIF8_BF16>, grid, st, src, n, n_vec, accum, d_amax_out); break;
        default: launch_pdl(amax_kernel<HIF8_F16>, grid, st, src, n, n_vec, accum, d_amax_out); break;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

int check_common(int dtype, int rnd, unsigned flags)
{
    if (dtype != HIF8_F32 && dtype != HIF8_BF16 && dtype != HIF8_F16) return HIF8_ERR_DTYPE;
    if (rnd < HIF8_RND_TA || rnd > HIF8_RND_SR) return HIF8_ERR_ROUND;
    if (flags & ~(HIF8_FLAG_SATURATE | HIF8_FLAG_NAN_TO_ZERO)) return HIF8_ERR_FLAGS;
    return HIF8_OK;
}

constexpr size_t kConvWorkspaceBytes = 256;

}  // namespace

int checked_device(int* sms) { return device_info(sms); }

}  // namespace hif8

using namespace hif8;

extern "C" {

int hif8_encode(const void* src, int src_dtype, uint8_t* dst, size_t n, int scale_exp, int rnd, unsigned flags,
                uint64_t seed, hif8_stream_t stream)
{
    int rc = check_common(src_dtype, rnd, flags);
    if (rc) return rc;
    if (scale_exp < -126 || scale_exp > 126) return HIF8_ERR_SCALE_RANGE;
    if (n == 0) return HIF8_OK;
    if (!src || !dst) return HIF8_ERR_NULL;
    if (ranges_overlap(src, n * dtype_bytes(src_dtype), dst, n)) return HIF8_ERR_OVERLAP;
    int sms; rc = device_info(&sms);
    if (rc) return rc;
    ConvParams p{};
    p.src = src; p.dst = dst; p.n = n; p.scale_exp = scale_exp; p.flags = flags; p.seed = seed;
    size_t out_align = src_dtype == HIF8_F32 ? 4 : 8;
    bool vec_ok = aligned16(src) && (reinterpret_cast<uintptr_t>(dst) % out_align) == 0;
    return dispatch_convert<false, false>(src_dtype, rnd, p, vec_ok, sms, (cudaStream_t)stream);
}

int hif8_encode_f32_patterns(uint32_t first_pattern, uint8_t* dst, size_t n, int scale_exp, int rnd, unsigned flags,
                             uint64_t seed, hif8_stream_t stream)
{
    int rc = check_common(HIF8_F32, rnd, flags);
    if (rc) return rc;
    if (scale_exp < -126 || scale_exp > 126) return HIF8_ERR_SCALE_RANGE;
    if (n > ((size_t)1 << 32)) return HIF8_ERR_SHAPE;
    if (n == 0) return HIF8_OK;
    if (!dst) return HIF8_ERR_NULL;
    int sms; rc = device_info(&sms);
    if (rc) return rc;
    ConvParams p{};
    p.dst = dst; p.n = n; p.scale_exp = scale_exp; p.flags = flags; p.seed = seed; p.pattern_first = first_pattern;
    const unsigned long long n_vec = (reinterpret_cast<uintptr_t>(dst) & 3u) ? 0 : n / 4;
    const unsigned grid = grid_for(n_vec, n, sms, kUnroll, kGroupsConvert);
    cudaStream_t st = (cudaStream_t)stream;
    switch (rnd) {
        case HIF8_RND_TA: launch_pdl(convert_kernel<HIF8_F32, HIF8_RND_TA, false, false, true>, grid, st, p, n_vec); break;
        case HIF8_RND_HR: launch_pdl(convert_kernel<HIF8_F32, HIF8_RND_HR, false, false, true>, grid, st, p, n_vec); break;
        case HIF8_RND_SSR: launch_pdl(convert_kernel<HIF8_F32, HIF8_RND_SSR, false, false, true>, grid, st, p, n_vec); break;
        case HIF8_RND_TE: launch_pdl(convert_kernel<HIF8_F32, HIF8_RND_TE, false, false, true>, grid, st, p, n_vec); break;
        default: launch_pdl(convert_kernel<HIF8_F32, HIF8_RND_SR, false, false, true>, grid, st, p, n_vec); break;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

int hif8_decode(const uint8_t* src, void* dst, int dst_dtype, size_t n, int scale_exp, hif8_stream_t stream)
{
    if (dst_dtype != HIF8_F32 && dst_dtype != HIF8_BF16 && dst_dtype != HIF8_F16) return HIF8_ERR_DTYPE;
    if (scale_exp < -126 || scale_exp > 126) return HIF8_ERR_SCALE_RANGE;
    if (n == 0) return HIF8_OK;
    if (!src || !dst) return HIF8_ERR_NULL;
    if (ranges_overlap(src, n, dst, n * dtype_bytes(dst_dtype))) return HIF8_ERR_OVERLAP;
    int sms; int rc = device_info(&sms);
    if (rc) return rc;
    unsigned long long pv = dst_dtype == HIF8_F32 ? 4 : 8;
    bool vec_ok = aligned16(dst) && (reinterpret_cast<uintptr_t>(src) % pv) == 0;
    unsigned long long n_vec = vec_ok ? n / pv : 0;
    unsigned grid = grid_for(n_vec, n, sms);
    cudaStream_t st = (cudaStream_t)stream;
    switch (dst_dtype) {
        case HIF8_F32: launch_pdl(decode_kernel<HIF8_F32>, grid, st, src, dst, n, n_vec, scale_exp); break;
        case HIF8_BF16: launch_pdl(decode_kernel<HIF8_BF16>, grid, st, src, dst, n, n_vec, scale_exp); break;
        default: launch_pdl(decode_kernel<HIF8_F16>, grid, st, src, dst, n, n_vec, scale_exp); break;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

// shared by hif8_amax_scale_encode and hif8_fake_quant
static int scaled_convert(bool fq, const void* src, void* dst, int dtype, size_t n, bool jit, int target_exp,
                          const int* d_scale_exp_in, int scale_exp, int rnd, unsigned flags, uint64_t seed,
                          float* d_amax_out, int* d_scale_exp_out, float* d_scale_out, void* workspace,
                          size_t workspace_bytes, bool want_amax, cudaStream_t st, void* scale_state = nullptr)
{
    int sms; int rc = device_info(&sms);
    if (rc) return rc;
    uint32_t* ws = reinterpret_cast<uint32_t*>(workspace);
    ConvParams p{};
    p.src = src; p.dst = dst; p.n = n; p.flags = flags; p.seed = seed; p.target_exp = target_exp;
    p.scale_exp = scale_exp; p.d_scale_exp = d_scale_exp_in;
    p.d_amax_out = d_amax_out; p.d_scale_exp_out = d_scale_exp_out; p.d_scale_out = d_scale_out;
    size_t out_align = fq ? 16 : (dtype == HIF8_F32 ? 4 : 8);
    bool vec_ok = aligned16(src) && (reinterpret_cast<uintptr_t>(dst) % out_align) == 0;
    if (jit || want_amax) {
        if (!ws || workspace_bytes < kConvWorkspaceBytes || (reinterpret_cast<uintptr_t>(ws) & 255u)) return HIF8_ERR_WORKSPACE;
        // (a delayed-scaling state keeps its two words at zero between passes itself)
        if (!scale_state) {
            if (launch_pdl(clear_accum_kernel, 1u, st, ws) != cudaSuccess) return HIF8_ERR_CUDA;
            g_launches.fetch_add(1, std::memory_order_relaxed);
        }
    }
    p.scale_state = scale_state;
    const bool inplace_fq = fq && !want_amax && ((rnd == HIF8_RND_TA && (dtype == HIF8_F32 || dtype == HIF8_BF16)) ||
                                                ((rnd == HIF8_RND_HR || rnd == HIF8_RND_SSR || rnd == HIF8_RND_TE || rnd == HIF8_RND_SR) && dtype == HIF8_BF16));
    if (jit) {
        rc = launch_amax(src, dtype, n, ws, nullptr, sms, st);
        if (rc) return rc;
        p.d_amax_bits = ws;
        p.reverse = 1;  // the amax pass has just read the tensor front to back
        if (inplace_fq) return launch_fq_ta(dtype, rnd, p, vec_ok, sms, st);
        return fq ? dispatch_convert<true, false>(dtype, rnd, p, vec_ok, sms, st)
                  : dispatch_convert<false, false>(dtype, rnd, p, vec_ok, sms, st);
    }
    if (inplace_fq) return launch_fq_ta(dtype, rnd, p, vec_ok, sms, st);
    if (want_amax) {
        p.amax_accum = ws;
        return fq ? dispatch_convert<true, true>(dtype, rnd, p, vec_ok, sms, st)
                  : dispatch_convert<false, true>(dtype, rnd, p, vec_ok, sms, st);
    }
    return fq ? dispatch_convert<true, false>(dtype, rnd, p, vec_ok, sms, st)
              : dispatch_convert<false, false>(dtype, rnd, p, vec_ok, sms, st);
}

int hif8_amax_scale_encode(const void* src, int src_dtype, uint8_t* dst, size_t n, int target_exp, int rnd,
                           unsigned flags, uint64_t seed, const int* d_scale_exp_in, float* d_amax_out,
                           int* d_scale_exp_out, float* d_scale_out, void* workspace, size_t workspace_bytes,
                           hif8_stream_t stream)
{
    int rc = check_common(src_dtype, rnd, flags);
    if (rc) return rc;
    if (target_exp < -22 || target_exp > 15) return HIF8_ERR_SCALE_RANGE;
    if (!workspace || workspace_bytes < kConvWorkspaceBytes || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return HIF8_ERR_WORKSPACE;
    if (n && (!src || !dst)) return HIF8_ERR_NULL;
    if (ranges_overlap(src, n * dtype_bytes(src_dtype), dst, n)) return HIF8_ERR_OVERLAP;
    bool jit = d_scale_exp_in == nullptr;
    return scaled_convert(false, src, dst, src_dtype, n, jit, target_exp, d_scale_exp_in, 0, rnd, flags, seed,
                          d_amax_out, d_scale_exp_out, d_scale_out, workspace, workspace_bytes, !jit,
                          (cudaStream_t)stream);
}

int hif8_amax(const void* src, int src_dtype, size_t n, float* d_amax_out, void* workspace, size_t workspace_bytes,
              hif8_stream_t stream)
{
    if (src_dtype != HIF8_F32 && src_dtype != HIF8_BF16 && src_dtype != HIF8_F16) return HIF8_ERR_DTYPE;
    if (!d_amax_out || (n && !src)) return HIF8_ERR_NULL;
    if (!workspace || workspace_bytes < kConvWorkspaceBytes || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return HIF8_ERR_WORKSPACE;
    int sms; int rc = device_info(&sms);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_pdl(clear_accum_kernel, 1u, st, reinterpret_cast<uint32_t*>(workspace)) != cudaSuccess) return HIF8_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_amax(src, src_dtype, n, reinterpret_cast<uint32_t*>(workspace), d_amax_out, sms, st);
}

int hif8_encode_from_amax(const void* src, int src_dtype, uint8_t* dst, size_t n, int target_exp, int rnd, unsigned flags,
                          uint64_t seed, const float* d_amax, int* d_scale_exp_out, float* d_scale_out, hif8_stream_t stream)
{
    int rc = check_common(src_dtype, rnd, flags);
    if (rc) return rc;
    if (target_exp < -22 || target_exp > 15) return HIF8_ERR_SCALE_RANGE;
    if (!d_amax || (n && (!src || !dst))) return HIF8_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(d_amax) & 3u) return HIF8_ERR_ALIGN;
    if (ranges_overlap(src, n * dtype_bytes(src_dtype), dst, n)) return HIF8_ERR_OVERLAP;
    int sms; rc = device_info(&sms);
    if (rc) return rc;
    ConvParams p{};
    p.src = src; p.dst = dst; p.n = n; p.flags = flags; p.seed = seed; p.target_exp = target_exp;
    p.d_amax_bits = reinterpret_cast<const uint32_t*>(d_amax);  // a non-negative float: its bits order as the value
    p.reverse = 1;  // the caller has just reduced amax over this tensor (hif8_amax), front to back
    p.d_scale_exp_out = d_scale_exp_out; p.d_scale_out = d_scale_out;
    const bool vec_ok = aligned16(src) && (reinterpret_cast<uintptr_t>(dst) % (src_dtype == HIF8_F32 ? 4 : 8)) == 0;
    return dispatch_convert<false, false>(src_dtype, rnd, p, vec_ok, sms, (cudaStream_t)stream);
}

int hif8_fake_quant(const void* src, void* dst, int dtype, size_t n, int use_amax, int scale_or_target_exp, int rnd,
                    unsigned flags, uint64_t seed, float* d_amax_out, int* d_scale_exp_out, void* workspace,
                    size_t workspace_bytes, hif8_stream_t stream)
{
    int rc = check_common(dtype, rnd, flags);
    if (rc) return rc;
    if (use_amax) {
        if (scale_or_target_exp < -22 || scale_or_target_exp > 15) return HIF8_ERR_SCALE_RANGE;
        if (!workspace || workspace_bytes < kConvWorkspaceBytes || (reinterpret_cast<uintptr_t>(workspace) & 255u))
            return HIF8_ERR_WORKSPACE;
    } else if (scale_or_target_exp < -126 || scale_or_target_exp > 126) return HIF8_ERR_SCALE_RANGE;
    if (n && (!src || !dst)) return HIF8_ERR_NULL;
    // in place (the same pointer) is allowed; any other sharing of bytes is not
    if (src != dst && ranges_overlap(src, n * dtype_bytes(dtype), dst, n * dtype_bytes(dtype))) return HIF8_ERR_OVERLAP;
    if (n == 0 && !use_amax) return HIF8_OK;
    return scaled_convert(true, src, dst, dtype, n, use_amax != 0, scale_or_target_exp, nullptr,
                          use_amax ? 0 : scale_or_target_exp, rnd, flags, seed, d_amax_out, d_scale_exp_out, nullptr,
                          workspace, workspace_bytes, false, (cudaStream_t)stream);
}

size_t hif8_workspace_bytes(int which, size_t n)
{
    switch (which) {
        case HIF8_WS_AMAX_SCALE_ENCODE:
        case HIF8_WS_FAKE_QUANT: return kConvWorkspaceBytes;
        case HIF8_WS_GEMM: return n ? 256 + 512 + 2 * n : 256;  // status word (+ both operands as BF16)
        default: return 0;
    }
}

const char* hif8_status_string(int status)
{
    switch (status) {
        case HIF8_OK: return "ok";
        case HIF8_ERR_NULL: return "required pointer is NULL";
        case HIF8_ERR_DTYPE: return "unknown element format";
        case HIF8_ERR_ROUND: return "unknown rounding method";
        case HIF8_ERR_FLAGS: return "unknown option bits";
        case HIF8_ERR_SCALE_RANGE: return "scale or target exponent out of range";
        case HIF8_ERR_SHAPE: return "unsupported extent or leading dimension";
        case HIF8_ERR_ALIGN: return "operand not 16-byte aligned";
        case HIF8_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case HIF8_ERR_CUDA: return "CUDA call failed or device is not compute capability 10.0";
        case HIF8_ERR_DEVICE_TIMEOUT: return "bounded device-side wait gave up";
        case HIF8_ERR_OVERLAP: return "source and destination share bytes";
        default: return "unknown status";
    }
}

uint64_t hif8_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Variant of hif8_amax_scale_encode for callers that have no workspace to give.
// The 8 bytes the amax reduction needs (running maximum + block ticket) live in a file-scope device array
// that every device loading this library carries until the process exits.
// ------------------------------------------------------------------------------------------------
namespace {
constexpr size_t kStaticScratchBytes = 256;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
// Device address of g_static_scratch per device ordinal.  In host code the array's name is only a handle for
// the runtime, not an address a kernel may dereference; the real address comes from cudaGetSymbolAddress.
std::atomic<void*> g_static_scratch_addr[64];
static_assert(kStaticScratchBytes == HIF8_STATIC_SCRATCH_BYTES, "the header states the size of the array");
static_assert(kStaticScratchBytes >= kConvWorkspaceBytes, "the array stands in for the conversion workspace");

int static_scratch(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HIF8_ERR_CUDA;
    void* ptr = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return HIF8_ERR_CUDA;
        g_static_scratch_addr[dev].store(ptr, std::memory_order_release);  // racing first callers store the same value
    }
    *out = ptr;
    return HIF8_OK;
}
}  // namespace

extern "C" int hif8_amax_scale_encode_static(const void* src, int src_dtype, uint8_t* dst, size_t n, int target_exp,
                                             int rnd, unsigned flags, uint64_t seed, const int* d_scale_exp_in,
                                             float* d_amax_out, int* d_scale_exp_out, float* d_scale_out,
                                             hif8_stream_t stream)
{
    int rc = check_common(src_dtype, rnd, flags);
    if (rc) return rc;
    if (target_exp < -22 || target_exp > 15) return HIF8_ERR_SCALE_RANGE;
    if (n > HIF8_STATIC_MAX_ELEMENTS) return HIF8_ERR_SHAPE;
    if (n && (!src || !dst)) return HIF8_ERR_NULL;
    if (ranges_overlap(src, n * dtype_bytes(src_dtype), dst, n)) return HIF8_ERR_OVERLAP;
    void* scratch = nullptr;
    rc = static_scratch(&scratch);
    if (rc) return rc;
    bool jit = d_scale_exp_in == nullptr;
    // scaled_convert clears the two words that must start at zero before the first kernel reads them
    return scaled_convert(false, src, dst, src_dtype, n, jit, target_exp, d_scale_exp_in, 0, rnd, flags, seed,
                          d_amax_out, d_scale_exp_out, d_scale_out, scratch, kStaticScratchBytes, !jit,
                          (cudaStream_t)stream);
}

// ------------------------------------------------------------------------------------------------
// Delayed scaling: the every-N-iterations amax cadence of Section 5.1 with a ring of past amax values.
// State (device memory, HIF8_SCALE_STATE_BYTES): bytes 0-255 the ScaleState record, bytes 256-511 the scratch of the
// conversion kernel's amax reduction (kept at zero between measuring passes by the kernel itself).
// ------------------------------------------------------------------------------------------------
namespace hif8 {
namespace {
__global__ void scale_state_init_kernel(ScaleState* st, int hist_len)
{
    const int i = threadIdx.x;
    if (i == 0) { st->scale_exp = 0; st->pos = 0; st->filled = 0; st->hist_len = hist_len; st->amax_last = 0.f; }
    if (i < HIF8_SCALE_HISTORY_MAX) st->ring[i] = 0.f;
    if (i < 2) reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(st) + 256)[i] = 0u;  // amax accumulator, block ticket
}

}  // namespace
}  // namespace hif8

extern "C" int hif8_scale_state_init(void* d_state, int hist_len, hif8_stream_t stream)
{
    if (!d_state) return HIF8_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(d_state) & 255u) return HIF8_ERR_WORKSPACE;
    if (hist_len < 1 || hist_len > HIF8_SCALE_HISTORY_MAX) return HIF8_ERR_SHAPE;
    int sms; int rc = device_info(&sms);
    if (rc) return rc;
    scale_state_init_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(reinterpret_cast<ScaleState*>(d_state), hist_len);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

extern "C" int hif8_delayed_scale_encode(const void* src, int src_dtype, uint8_t* dst, size_t n, int rnd, unsigned flags,
                                         uint64_t seed, void* d_state, int measure, int target_exp, hif8_stream_t stream)
{
    int rc = check_common(src_dtype, rnd, flags);
    if (rc) return rc;
    if (target_exp < -22 || target_exp > 15) return HIF8_ERR_SCALE_RANGE;
    if (!d_state || (n && (!src || !dst))) return HIF8_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(d_state) & 255u) return HIF8_ERR_WORKSPACE;
    if (ranges_overlap(src, n * dtype_bytes(src_dtype), dst, n)) return HIF8_ERR_OVERLAP;
    ScaleState* state = reinterpret_cast<ScaleState*>(d_state);
    cudaStream_t st = (cudaStream_t)stream;
    if (!measure)  // conversion alone, exponent read from the state on the device
        return scaled_convert(false, src, dst, src_dtype, n, false, target_exp, &state->scale_exp, 0, rnd, flags, seed, nullptr,
                              nullptr, nullptr, nullptr, 0, false, st);
    // one pass: convert with the exponent in force and reduce amax; the last block to finish pushes it into the ring and
    // sets the exponent for the next conversion
    return scaled_convert(false, src, dst, src_dtype, n, false, target_exp, &state->scale_exp, 0, rnd, flags, seed,
                          &state->amax_last, nullptr, nullptr, reinterpret_cast<unsigned char*>(d_state) + 256, kConvWorkspaceBytes,
                          true, st, d_state);
}
