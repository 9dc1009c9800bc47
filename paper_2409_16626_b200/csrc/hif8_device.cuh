// Device-side building blocks of the conversion kernels, shared by the translation units that convert: field packing
// and the compile-time round-half-away table (Tables 1-3), byte -> binary32 (Eq. 1, Eq. 2), Philox4x32-10, the
// per-element encoder for every rounding mode of Section 3, shared-memory table set-up, scale and amax helpers.
// Everything lives in an unnamed namespace: each translation unit gets its own copy.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "hif8.h"

namespace hif8 {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;
constexpr int kBlocksPerSM = 8;

// ------------------------------------------------------------------------------------------------
// Field packing (Table 1: sign | dot | exponent | mantissa; Table 2 prefix code; Table 3 exponent ranges)
// ------------------------------------------------------------------------------------------------
__host__ __device__ constexpr int mant_width(int E)
{
    int a = E < 0 ? -E : E;
    return (E <= -16) ? 0 : (a <= 3 ? 3 : (a <= 7 ? 2 : 1));
}

// magnitude byte (bit 7 clear) of 2^E * 1.M, E in [-22, 15], M already `mant_width(E)` bits wide
__host__ __device__ constexpr uint32_t pack_magnitude(int E, uint32_t M)
{
    if (E <= -16) return (uint32_t)(E + 23);  // Eq. 2: denormal, mantissa field = E + 23
    uint32_t a = (uint32_t)(E < 0 ? -E : E), se = E < 0 ? 1u : 0u;
    if (a == 0) return 0x08u | M;                                     // dot 0001
    if (a == 1) return 0x10u | (se << 3) | M;                         // dot 001, Em = {Se}
    if (a <= 3) return 0x20u | (se << 4) | ((a & 1u) << 3) | M;       // dot 01,  Em = {Se, Mag[2]}
    if (a <= 7) return 0x40u | (se << 4) | ((a & 3u) << 2) | M;       // dot 10,  Em = {Se, Mag[2:3]}
    return 0x60u | (se << 4) | ((a & 7u) << 1) | M;                   // dot 11,  Em = {Se, Mag[2:4]}
}

// Round-half-away result for the binary32 patterns whose top 13 bits are `idx`
// (1 sign, 8 exponent, 4 mantissa bits).
__host__ __device__ constexpr uint8_t ta_entry(uint32_t idx)
{
    uint32_t sign = (idx >> 12) << 7;
    int e = (int)((idx >> 4) & 0xFF);
    uint32_t m4 = idx & 0xF;
    if (e == 255) return m4 ? (uint8_t)0x80 : (uint8_t)(sign | 0x6F);   // NaN (canonical has m4 = 15) / Inf
    int E = e - 127;
    if (E >= 16) return (uint8_t)(sign | 0x6F);
    if (E <= -24) return 0;                       // below half of 2^-22: the single zero pattern
    if (E == -23) return (uint8_t)(sign | 0x01);  // [2^-23, 2^-22) rounds up to 2^-22 (tie away)
    int w = mant_width(E);
    uint32_t M = m4 >> (4 - w);
    uint32_t rbit = (m4 >> (3 - w)) & 1u;         // MSB of the discarded bits
    M += rbit;
    if (M == (1u << w)) { M = 0; E += 1; }        // carry into the exponent; the mantissa is then zero
    if (E >= 16) return (uint8_t)(sign | 0x6F);
    return (uint8_t)(sign | pack_magnitude(E, M));  // E = 15, M = 1 is the Inf pattern by construction
}

// Truncating companion of ta_entry, for patterns that a threshold-based rounding has already rounded: the mantissa bits
// beyond the binade's width are ignored instead of rounded.  Two binades below the format's range keep the meaning the
// threshold modes give them after their own carry trick: 2^-23 stands for "reached the threshold" (-> 2^-22), anything
// smaller for zero.
__host__ __device__ constexpr uint8_t trunc_entry(uint32_t idx)
{
    uint32_t sign = (idx >> 12) << 7;
    int e = (int)((idx >> 4) & 0xFF);
    uint32_t m4 = idx & 0xF;
    if (e == 255) return m4 ? (uint8_t)0x80 : (uint8_t)(sign | 0x6F);
    int E = e - 127;
    if (E >= 16) return (uint8_t)(sign | 0x6F);
    if (E <= -24) return 0;
    if (E == -23) return (uint8_t)(sign | 0x01);
    return (uint8_t)(sign | pack_magnitude(E, m4 >> (4 - mant_width(E))));  // E = 15, M = 1 is the Inf pattern by construction
}

struct TaTable { uint8_t v[8192]; };
constexpr TaTable make_ta_table()
{
    TaTable t{};
    for (uint32_t i = 0; i < 8192; i++) t.v[i] = ta_entry(i);
    return t;
}
__device__ const TaTable g_ta_table = make_ta_table();
constexpr TaTable make_trunc_table()
{
    TaTable t{};
    for (uint32_t i = 0; i < 8192; i++) t.v[i] = trunc_entry(i);
    return t;
}
__device__ const TaTable g_trunc_table = make_trunc_table();

// Hybrid / simplified stochastic rounding (Section 3.2, Eq. 3): both neighbours of a scaled magnitude in one word.  Index =
// (biased exponent, top three mantissa bits) of the magnitude, no sign: 2^-23 .. 2^16 are the binades that differ.
//   bits 0-4   left shift that puts the discarded field of this binade at the top of a word (9 + mantissa width)
//   bits 8-15  the neighbour below (truncation), bits 16-23 the neighbour above; bit 7 of either byte says "takes the
//              sign" (clear for the single zero; the NaN pattern 0x80 reads as a zero magnitude that takes a sign which
//              the caller arranges to be set)
//   bits 30-31 are filled in at set-up (stochastic or round-half-away binade)
// The binade of 2^-23 stands for everything below 2^-22 (see pair32_lookup): neighbours 0 and 2^-22, no mantissa bit kept.
__host__ __device__ constexpr uint32_t pair_entry(uint32_t idx)
{
    int e = (int)(idx >> 3);
    uint32_t m3 = idx & 7u;
    if (e == 255) return m3 ? 0x00808009u : 0x00EFEF09u;  // NaN / Inf
    int E = e - 127;
    if (E >= 16) return 0x00EFEF09u;
    if (E < -23) return 0u;
    if (E == -23) return 0x00810009u;
    int w = mant_width(E);
    uint32_t M = m3 >> (3 - w);
    uint32_t down = pack_magnitude(E, M);  // E = 15, M = 1 is the Inf pattern by construction
    uint32_t up = (M + 1u == (1u << w)) ? (E + 1 >= 16 ? 0x6Fu : pack_magnitude(E + 1, 0u)) : pack_magnitude(E, M + 1u);
    return (uint32_t)(9 + w) | ((down | 0x80u) << 8) | ((up | 0x80u) << 16);
}
struct PairTable { uint32_t v[2048]; };
constexpr PairTable make_pair_table()
{
    PairTable t{};
    for (uint32_t i = 0; i < 2048; i++) t.v[i] = pair_entry(i);
    return t;
}
__device__ const PairTable g_pair_table = make_pair_table();

// value of one byte as binary32 bits (Eq. 1 / Eq. 2 / specials)
__device__ __forceinline__ uint32_t decode_bits_f32(uint32_t c)
{
    uint32_t sign = (c & 0x80u) << 24, m = c & 0x7Fu;
    if (m == 0) return sign ? 0x7FC00000u : 0u;
    if (m == 0x6F) return sign | 0x7F800000u;
    if (m < 8) return sign | ((m + 104u) << 23);  // 2^(m-23)
    int E; uint32_t M, w;
    if (m < 0x10)      { E = 0; M = m & 7; w = 3; }
    else if (m < 0x20) { E = 1; M = m & 7; w = 3; if (m & 0x08) E = -E; }
    else if (m < 0x40) { E = 2 | ((m >> 3) & 1); M = m & 7; w = 3; if (m & 0x10) E = -E; }
    else if (m < 0x60) { E = 4 | ((m >> 2) & 3); M = m & 3; w = 2; if (m & 0x10) E = -E; }
    else               { E = 8 | ((m >> 1) & 7); M = m & 1; w = 1; if (m & 0x10) E = -E; }
    return sign | ((uint32_t)(E + 127) << 23) | (M << (23 - w));
}

// ------------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): counter (c0, c1, 0, 0), key (k0, k1)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t k0, uint32_t k1)
{
    uint32_t x0 = c0, x1 = c1, x2 = 0, x3 = 0;
#pragma unroll
    for (int r = 0; r < 10; r++) {
        uint32_t hi0 = __umulhi(0xD2511F53u, x0), lo0 = 0xD2511F53u * x0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, x2), lo1 = 0xCD9E8D57u * x2;
        uint32_t n0 = hi1 ^ x1 ^ k0, n2 = hi0 ^ x3 ^ k1;
        x0 = n0; x1 = lo1; x2 = n2; x3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return make_uint4(x0, x1, x2, x3);
}

// word `lane` (0..3) of a Philox block, picked with selects (an array indexed by a variable would live in local memory)
__device__ __forceinline__ uint32_t philox_word(const uint4& r, unsigned lane)
{
    const uint32_t lo = (lane & 1u) ? r.y : r.x, hi = (lane & 1u) ? r.w : r.z;
    return (lane & 2u) ? hi : lo;
}

// ------------------------------------------------------------------------------------------------
// Programmatic dependent launch.  Every kernel here is launched so that it may be scheduled while the previous
// kernel of the stream is still draining: it signals its own dependents at once (they can only start after all of
// this grid's blocks have started), does the work that touches no global input (table set-up), and waits for the
// previous grid to have completed and flushed before its first global read or write.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------------------------------------
// Scale handling
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int clamp_exp(int e) { return e < -126 ? -126 : (e > 126 ? 126 : e); }
__device__ __forceinline__ float pow2f(int e) { return __uint_as_float((uint32_t)(e + 127) << 23); }  // |e| <= 126

// scale exponent from the bits of amax (a non-negative finite binary32)
__device__ __forceinline__ int scale_exp_from_amax(uint32_t ab, int target_exp)
{
    if (ab == 0) return 0;
    int e = (ab >> 23) ? (int)(ab >> 23) - 127 : (31 - __clz(ab)) - 149;  // floor(log2 amax)
    return clamp_exp(target_exp - e);
}

struct ConvParams {
    const void* src;
    void* dst;
    unsigned long long n;
    int scale_exp;                // used when neither pointer below is set
    const int* d_scale_exp;       // delayed scaling: exponent read from the device
    const uint32_t* d_amax_bits;  // just-in-time scaling: exponent derived from this amax
    int target_exp;
    unsigned flags;
    unsigned long long seed;
    uint32_t* amax_accum;         // when the kernel also reduces amax: accumulator and ticket (2 words)
    float* d_amax_out;
    int* d_scale_exp_out;
    float* d_scale_out;
    void* scale_state;            // delayed scaling: ScaleState that the last block of an amax-reducing pass advances
    uint32_t pattern_first;       // PATTERN kernels only: element i is the FP32 value whose encoding is pattern_first + i
    int reverse;                  // walk the tensor from its end: set for the second pass of just-in-time scaling, so that
                                  // the lines the amax pass read last (still in L2) are the ones re-read first
};

template <int SRC> struct SrcTraits;
template <> struct SrcTraits<HIF8_F32>  { static constexpr int kPerVec = 4; };
template <> struct SrcTraits<HIF8_BF16> { static constexpr int kPerVec = 8; };
template <> struct SrcTraits<HIF8_F16>  { static constexpr int kPerVec = 8; };

// element k of a 16-byte source vector: its value as binary32 and its raw encoding
template <int SRC>
__device__ __forceinline__ void unpack(const uint4& v, int k, float& x, uint32_t& raw)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (SRC == HIF8_F32) { raw = w[k]; x = __uint_as_float(raw); }
    else {
        uint32_t word = w[k >> 1];
        raw = (k & 1) ? (word >> 16) : (word & 0xFFFFu);
        if (SRC == HIF8_BF16) x = __uint_as_float(raw << 16);
        else x = __half2float(__ushort_as_half((unsigned short)raw));
    }
}

template <int SRC>
__device__ __forceinline__ void load_scalar(const void* p, unsigned long long i, float& x, uint32_t& raw)
{
    if (SRC == HIF8_F32) { raw = reinterpret_cast<const uint32_t*>(p)[i]; x = __uint_as_float(raw); }
    else {
        raw = reinterpret_cast<const unsigned short*>(p)[i];
        if (SRC == HIF8_BF16) x = __uint_as_float(raw << 16);
        else x = __half2float(__ushort_as_half((unsigned short)raw));
    }
}

// binary32 value -> encoding of the destination format, round to nearest even
template <int DT> __device__ __forceinline__ uint32_t to_bits(float v)
{
    if (DT == HIF8_F32) return (v != v) ? 0x7FC00000u : __float_as_uint(v);
    if (DT == HIF8_BF16) {
        if (v != v) return 0x7FC0u;
        return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v));
    }
    if (v != v) return 0x7E00u;
    return (uint32_t)__half_as_ushort(__float2half_rn(v));
}

// ------------------------------------------------------------------------------------------------
// One element: scaled value -> HiF8 byte
// ------------------------------------------------------------------------------------------------
// Rounding table thr[], indexed by the biased exponent of the scaled value (never by its sign: values of either sign would
// otherwise hit different words of the same bank).
//  * SR: thr[e] = sh, the number of discarded mantissa bits (23 - width; 0: nothing to round).
//  * TE: thr[e] = half - 1 (bits 0-22; half itself where no mantissa bit is kept: the implicit one is odd), bit 26 "add
//    the kept LSB", sh in bits 27-31; the binade of 2^-23 adds 2^23 - 1 (anything above the tie carries into 2^-22).
//  * Hybrid / simplified stochastic rounding, FP32 sources: thr[] is not used.  One word per (exponent, top three
//    mantissa bits) holds both neighbours and the binade's shift (pair_entry); the discarded field, left-aligned, is
//    compared with the threshold (SR14: the source's low 14 bits; one half in the round-half-away binades of Eq. 3) and
//    the comparison picks the byte: one 4-byte lookup per element.  (The same form measured slower than the one below
//    for 16-bit sources: 54.7 against 41.7 us per 2^26 BF16 elements.)
//  * Hybrid / simplified stochastic rounding, 16-bit sources (T2 = 2 LSB + 1, complement 3 - 2 LSB): an increment is added
//    to the bit pattern so that the carry out of the discarded field rounds up (also across binade and width boundaries),
//    the old binade's discarded bits are cleared (~0 << sh) and the code is read from the truncating table.
//    thr[2e + LSB] = (3 - 2 LSB) * 2^(sh-2), or one half in a round-half-away binade, with sh in bits 0-4.  Below 2^-22
//    (result 0 or 2^-22, F = |y| / 2^-22) only the binades of 2^-23 and 2^-24 can reach the threshold; their entries add
//    the complement at the top of the pattern and step the exponent down by one / two, which leaves 2^-23 or 2^-22 when
//    the threshold is reached and something below 2^-23 when not.
// FP32 sources, hybrid / simplified stochastic rounding: the neighbour-pair word of the scaled value y and whether the
// upper neighbour is taken
template <int MODE>
__device__ __forceinline__ bool pair32_lookup(float y, uint32_t raw, const uint32_t* tab, uint32_t& ent)
{
    const float a = fabsf(y);
    // below 2^-22 the result is 0 or 2^-22 with F = |y| / 2^-22: |y| / 2 + 2^-23 with truncation puts floor(F 2^23)
    // into the mantissa of a value in the binade of 2^-23, and exceeds |y| exactly when |y| < 2^-22
    const uint32_t w = __float_as_uint(fmaxf(a, __fmaf_rz(a, 0.5f, 1.1920928955078125e-07f)));
    ent = tab[w >> 20];
    const uint32_t u = __funnelshift_l(0u, w, ent);  // discarded field, left-aligned (shift = low five bits of ent)
    uint32_t thr = max(raw << 18, 0x40000u);         // SR14: round up iff F14 >= max(T14, 1), T14 = low 14 source bits
    if (MODE == HIF8_RND_HR) {                       // round-half-away binades of Eq. 3 (bit 31): the top discarded bit decides
        const uint32_t m = (uint32_t)((int32_t)ent >> 31);
        thr = (thr & ~m) | (m & 0x80000000u);
    }
    return u >= thr;
}

// Round half away with the code table read sign-free.  The table's negative half lies 4096 bytes (a multiple of the
// 128-byte bank period) above the positive one, so +x and -x of one binade would always meet in one bank; reading the
// non-negative half only costs a warp about half the shared-memory wavefronts on zero-centred data.
__device__ __forceinline__ uint32_t ta_magnitude_code(float x, float scale, const uint8_t* s_ta)
{
    return s_ta[__float_as_uint(fabsf(x) * scale) >> 19];
}

// ... and the signs of a source vector's elements put back onto their packed magnitude codes (w0: elements 0-3, w1:
// elements 4-7 of a 16-bit source): bit 7 of every code that is not the single zero (code + 0x7F carries into bit 7 for
// 0x01 .. 0x80; NaN, 0x80, keeps its encoding either way).
template <int SRC>
__device__ __forceinline__ void put_signs(const uint4& v, uint32_t& w0, uint32_t& w1)
{
    if (SRC == HIF8_F32) {
        const uint32_t s = __byte_perm(__byte_perm(v.x, v.y, 0x0073u), __byte_perm(v.z, v.w, 0x0073u), 0x5410u);  // byte 3 of each word
        w0 |= (w0 + 0x7F7F7F7Fu) & s & 0x80808080u;
    } else {
        const uint32_t s0 = __byte_perm(v.x, v.y, 0x7531u), s1 = __byte_perm(v.z, v.w, 0x7531u);  // bytes 1 and 3 of each word
        w0 |= (w0 + 0x7F7F7F7Fu) & s0 & 0x80808080u;
        w1 |= (w1 + 0x7F7F7F7Fu) & s1 & 0x80808080u;
    }
}

template <int MODE, int SRC>
__device__ __forceinline__ uint32_t encode_one(float x, uint32_t raw, float scale, const uint8_t* s_ta,
                                               const uint32_t* s_thr, uint32_t word)
{
    constexpr bool kPair = (MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR) && SRC == HIF8_F32;
    const float y = kPair ? x * -scale : x * scale;
    uint32_t t = __float_as_uint(y);
    if (MODE == HIF8_RND_TA) return s_ta[t >> 19];

    if ((MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR) && SRC == HIF8_F32) {
        // s_ta holds the neighbour-pair words here (see pair_entry).  The scale was negated above: every sign is then
        // inverted except that of the canonical NaN the multiply produces, so "bit 7 of the code AND NOT the sign" gives
        // the sign of every finite / infinite result, a set bit for NaN and nothing for the single zero.
        uint32_t ent;
        const bool up = pair32_lookup<MODE>(y, raw, reinterpret_cast<const uint32_t*>(s_ta), ent);
        const uint32_t c = __byte_perm(ent, 0u, up ? 0x4442u : 0x4441u);
        return c & (~(t >> 24) | 0x7Fu);
    }
    if (MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR) {  // 16-bit sources; s_ta is the truncating table here
        // two entries per exponent, chosen by the source LSB, with sh in bits 0-4 (a widened 16-bit pattern has zeros
        // there, so they cannot carry)
        const uint32_t ent = s_thr[((t >> 22) & 0x1FEu) | (raw & 1u)];
        return s_ta[((t + ent) & (0xFFFFFFFFu << (ent & 31u))) >> 19];
    }

    if (MODE == HIF8_RND_TE) {
        // round half to even as one increment: half - 1 plus the kept LSB (the carry rounds up exactly when the discarded
        // field exceeds one half, or equals it with an odd kept significand); s_ta is the truncating table with 2^-23 -> 0
        const uint32_t ent = s_thr[(t >> 23) & 0xFFu];  // bits 0-22 constant, bit 26 "add the kept LSB", bits 27-31 sh
        const uint32_t sh = ent >> 27;
        const uint32_t lsb = (t >> sh) & (ent >> 26) & 1u;
        return s_ta[((t + (ent & 0x03FFFFFFu) + lsb) & (0xFFFFFFFFu << sh)) >> 19];
    }

    const bool sub = (t & 0x7FFFFFFFu) < 0x34800000u;  // |y| < 2^-22 (zero included): result is 0 or 2^-22
    // Below 2^-22 the kept bits are zero and the fraction is F = |y| / 2^-22.  Adding 2^-22 with truncation puts
    // floor(F 2^23) into the mantissa field of a value in the binade of 2^-22, so the common code rounds it like a
    // 0-bit-mantissa binade (result 2^-22 or 2^-21); it is moved down again afterwards.
    const uint32_t tz = __float_as_uint(__fadd_rz(fabsf(y), 2.384185791015625e-07f));

    // standard SR
    constexpr int kSrBits = (SRC == HIF8_F32) ? 24 : 16;
    const uint32_t sign7 = (t >> 24) & 0x80u;
    if (SRC == HIF8_F32 && sub) {
        // the 24-bit threshold is wider than a binary32 fraction: compare F24 = floor(|y| 2^46) directly
        const uint32_t f24 = __float2uint_rz(fabsf(y) * 70368744177664.f);
        return f24 >= max(word >> 8, 1u) ? (sign7 | 0x01u) : 0u;
    }
    t = sub ? (tz | (t & 0x80000000u)) : t;
    const uint32_t sh = s_thr[(t >> 23) & 0xFFu];  // discarded mantissa bits (23 - width); 0: nothing to round
    const uint32_t s = sh ? sh : 23u;
    // threshold T of Section 3.2, compared as max(T,1) so that a zero fraction never rounds up
    const uint32_t T = max(word >> (32 - kSrBits), 1u);
    uint32_t inc;
    if (SRC == HIF8_F32) {
        const uint32_t k = 24u - s;  // F24 = discarded << k; up iff discarded >= ceil(T / 2^k)
        inc = (1u << s) - ((T + (1u << k) - 1u) >> k);
    } else inc = (0x10000u - T) << (s - 16);
    if (sh == 0) inc = 0;
    const uint32_t tr = (t + inc) & (0xFFFFFFFFu << sh);
    uint32_t code = s_ta[tr >> 19];
    if (sub) code = ((code & 0x7Fu) == 0x02u) ? (sign7 | 0x01u) : 0u;  // 2^-21 -> 2^-22, 2^-22 -> the single zero
    return code;
}

// ------------------------------------------------------------------------------------------------
// BF16 sources, hybrid / simplified stochastic rounding in packed BF16 arithmetic (two elements per instruction, on the
// floating-point pipe).  SR2 rounds up iff F >= T2 / 4 with T2 = 2 LSB + 1, i.e. iff |y| + (1 - T2 / 4) ulp reaches the
// upper neighbour: add 0.75 ulp minus LSB * 0.5 ulp (0.5 ulp in a round-half-away binade of Eq. 3) and let a truncating
// code table drop what is left of the discarded bits.  The addend is a multiple of the 8-bit significand's grid, so the
// sum is exact unless it carries into the next binade, where the leftover is below one unit of any mantissa width.
//   inck[e] (by the biased exponent of |y|): low half the addend for LSB = 0, high half -(0.5 ulp) * 2^69
//   LSB term: the source's LSB as the BF16 pattern 0x0001 (2^-133) times 2^64, times the high half
//   Below 2^-22 (result 0 or 2^-22, F = |y| / 2^-22): the binades of 2^-23 and 2^-24 add 3 * 2^-24 - LSB * 2 * 2^-24 and
//   reach 2^-22 exactly when floor(4 F) >= T2; smaller values add nothing.  Anything that ends below 2^-22 reads zero.
//   code8[(e, top three mantissa bits)] is the truncated magnitude with bit 7 = "takes the sign" (see pair_entry).
// ------------------------------------------------------------------------------------------------
template <int MODE>
__device__ __forceinline__ void setup_sum16(uint8_t* code8, uint32_t* inck, unsigned flags)
{
    for (int i = threadIdx.x; i < 512; i += kThreads) {  // four codes per word
        uint32_t word = 0;
#pragma unroll
        for (int b = 0; b < 4; b++) {
            const int idx = 4 * i + b, e = idx >> 3;
            uint32_t c = 0;
            if (e >= 105 && e <= 142) c = (g_pair_table.v[idx] >> 8) & 0xFFu;
            else if (e > 142) c = (e == 255 && (idx & 7)) ? 0x80u : 0xEFu;
            if ((flags & HIF8_FLAG_SATURATE) && (c & 0x7Fu) == 0x6Fu) c &= 0xFEu;
            if ((flags & HIF8_FLAG_NAN_TO_ZERO) && c == 0x80u) c = 0u;
            word |= c << (8 * b);
        }
        reinterpret_cast<uint32_t*>(code8)[i] = word;
    }
    {
        const int e = threadIdx.x, E = e - 127;  // kThreads == 256 biased exponents
        uint32_t v = 0u;
        if (E >= -24 && E <= 15) {
            // h = biased exponent of 0.5 ulp; below 2^-22 the unit is 2^-22 whatever the binade
            const int h = (E < -22 ? -23 : E - mant_width(E) - 1) + 127;
            if (MODE == HIF8_RND_HR && E > -4 && E < 4) v = (uint32_t)h << 7;                       // 0.5 ulp, no LSB term
            else v = (((uint32_t)h << 7) | 0x40u) | ((0x8000u | ((uint32_t)(h + 69) << 7)) << 16);  // 0.75 ulp; -(0.5 ulp) 2^69
        }
        inck[e] = v;
    }
    __syncthreads();
}

// the negated power-of-two scale as two BF16 values
__device__ __forceinline__ uint32_t neg_scale_bf16x2(float scale) { return (0x8000u | (__float_as_uint(scale) >> 16)) * 0x00010001u; }

__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

__device__ __forceinline__ uint32_t fma_bf16x2(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// W: two source patterns, Y = W times the negated scale.  Returns the two codes before the sign step in bytes 0 and 1;
// the caller clears bit 7 of a code where bit 15 / 31 of Y is set.
__device__ __forceinline__ uint32_t encode_sum16(uint32_t W, uint32_t Y, const uint8_t* code8, const uint32_t* inck)
{
    const uint32_t A = Y & 0x7FFF7FFFu;
    const uint32_t el = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(inck) + ((A >> 5) & 0x3FCu));
    const uint32_t eh = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const char*>(inck) + ((A >> 21) & 0x3FCu));
    const uint32_t lsb = mul_bf16x2(W & 0x00010001u, 0x5F805F80u);  // LSB * 2^-133 * 2^64
    const uint32_t add = fma_bf16x2(lsb, __byte_perm(el, eh, 0x7632), __byte_perm(el, eh, 0x5410));
    const uint32_t R = fma_bf16x2(A, 0x3F803F80u, add);  // |y| + addend, non-negative
    return (uint32_t)code8[(R >> 4) & 0x7FFu] | ((uint32_t)code8[R >> 20] << 8);
}

// ------------------------------------------------------------------------------------------------
// Block set-up: tables into shared memory, scale
// ------------------------------------------------------------------------------------------------
struct __align__(16) SmemTables {
    uint8_t ta[8192];
    uint32_t thr[512];
    float dec[256];
};

template <bool NEED_TA, bool NEED_SH, bool NEED_DEC, int MODE = HIF8_RND_TA, int SRC = HIF8_F32>
__device__ __forceinline__ void setup_tables(SmemTables& s, unsigned flags)
{
    constexpr bool kPair = (MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR) && SRC == HIF8_F32;  // neighbour-pair words instead of code bytes
    if (NEED_TA && kPair) {
        // 2048 words indexed by (exponent, top three mantissa bits).  The magnitudes that reach the lookup lie in
        // 2^-23 .. Inf / NaN; 2^-23 .. 2^15 come from the compile-time table, everything above is Inf.
        uint32_t* d = reinterpret_cast<uint32_t*>(s.ta);
        for (int i = threadIdx.x; i < 2048; i += kThreads) {
            const int e = i >> 3, E = e - 127;
            uint32_t v = 0u;
            if (e >= 104 && e <= 142) v = g_pair_table.v[i];
            else if (e > 142) v = (e == 255 && (i & 7)) ? 0x00808009u : 0x00EFEF09u;
            if (flags) {  // Section 3 options: patch the Inf / NaN bytes
                uint32_t lo = (v >> 8) & 0xFFu, hi = (v >> 16) & 0xFFu;
                if (flags & HIF8_FLAG_SATURATE) {
                    if ((lo & 0x7Fu) == 0x6Fu) lo &= 0xFEu;
                    if ((hi & 0x7Fu) == 0x6Fu) hi &= 0xFEu;
                }
                if (flags & HIF8_FLAG_NAN_TO_ZERO) {
                    if (lo == 0x80u) lo = 0u;
                    if (hi == 0x80u) hi = 0u;
                }
                v = (v & 0xFF0000FFu) | (lo << 8) | (hi << 16);
            }
            // Eq. 3: round half away for |E| < 4 under hybrid rounding (bits 31-30 = 10), stochastic elsewhere (01)
            v |= (MODE == HIF8_RND_HR && E > -4 && E < 4) ? 0x80000000u : 0x40000000u;
            d[i] = v;
        }
    }
    if (NEED_TA && !kPair) {
        // Only binades 2^-24 .. 2^16 differ from their neighbours: those 41 x 16 entries per sign come from the
        // compile-time table (1.3 KiB of global reads per block); everything below is zero, everything above is
        // Inf (or NaN in the all-ones exponent), written straight into shared memory.
        constexpr bool kTrunc = MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR || MODE == HIF8_RND_TE;  // modes that round before the lookup
        const uint4* g = reinterpret_cast<const uint4*>(kTrunc ? g_trunc_table.v : g_ta_table.v);
        uint4* d = reinterpret_cast<uint4*>(s.ta);
        for (int i = threadIdx.x; i < 512; i += kThreads) {
            const uint32_t e = i & 255, inf = ((uint32_t)(i >> 8) << 7) | 0x6Fu;
            uint4 v;
            if (e < 103) v = make_uint4(0, 0, 0, 0);
            else if (MODE == HIF8_RND_TE && e == 104) v = make_uint4(0, 0, 0, 0);  // TE: what is left in the binade of 2^-23 is the exact tie
            else if (e <= 143) v = g[i];
            else if (e < 255) { uint32_t w = inf * 0x01010101u; v = make_uint4(w, w, w, w); }
            else v = make_uint4(0x80808000u | inf, 0x80808080u, 0x80808080u, 0x80808080u);
            if (flags) {  // Section 3 options: patch the Inf / NaN entries
                uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    uint32_t o = 0;
#pragma unroll
                    for (int b = 0; b < 4; b++) {
                        uint32_t c = (w[j] >> (8 * b)) & 0xFFu;
                        if ((flags & HIF8_FLAG_SATURATE) && (c & 0x7Fu) == 0x6Fu) c &= 0xFEu;
                        if ((flags & HIF8_FLAG_NAN_TO_ZERO) && c == 0x80u) c = 0;
                        o |= c << (8 * b);
                    }
                    w[j] = o;
                }
                v = make_uint4(w[0], w[1], w[2], w[3]);
            }
            d[i] = v;
        }
    }
    if (NEED_SH && !kPair) {
        const int e = threadIdx.x, E = e - 127;  // kThreads == 256 biased exponents
        constexpr bool kThreshold = MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR;
        // TE / SR: thr[e] = e0.  Threshold modes (16-bit sources): thr[2e] = e0 (source LSB 0), thr[2e + 1] = e1 (LSB 1).
        uint32_t e0 = 0, e1 = 0;
        if (E < 16 && E >= -22) {
            const uint32_t sh = 23u - (uint32_t)mant_width(E);
            const bool stochastic = MODE == HIF8_RND_SSR || E <= -4 || E >= 4;  // Eq. 3 for HR
            if (MODE == HIF8_RND_TE) e0 = (sh == 23u ? (1u << 22) : ((1u << (sh - 1u)) - 1u) | (1u << 26)) | (sh << 27);
            else if (!kThreshold) e0 = sh;  // SR: only the width is read
            else if (stochastic) { e0 = (3u << (sh - 2u)) | sh; e1 = (1u << (sh - 2u)) | sh; }  // complement 3 - 2 LSB
            else e0 = e1 = (1u << (sh - 1u)) | sh;
        } else if (MODE == HIF8_RND_TE && E == -23) {
            e0 = ((1u << 23) - 1u) | (23u << 27);  // above 2^-23 -> carry -> 2^-22; exactly 2^-23 stays (-> 0 in TE's table)
        } else if (kThreshold && (E == -23 || E == -24)) {
            const uint32_t j = (uint32_t)(-23 - E);  // complement << (22 + j), then j + 1 binades down
            e0 = ((3u << (22u + j)) - ((j + 1u) << 23)) | 23u;
            e1 = ((1u << (22u + j)) - ((j + 1u) << 23)) | 23u;
        }
        if (kThreshold) { s.thr[2 * e] = e0; s.thr[2 * e + 1] = e1; }
        else s.thr[e] = e0;
    }
    if (NEED_DEC) s.dec[threadIdx.x] = __uint_as_float(decode_bits_f32(threadIdx.x));
    __syncthreads();
}

// Delayed scaling (the every-N-iterations amax cadence of Section 5.1): exponent in force and a ring of past amax values
struct ScaleState {
    int scale_exp;  // exponent in force
    int pos;        // next ring slot
    int filled;     // valid ring entries
    int hist_len;
    float amax_last;
    int pad[3];
    float ring[HIF8_SCALE_HISTORY_MAX];
};
static_assert(sizeof(ScaleState) <= 256, "state record too large");

// push the amax just measured (bit pattern of a non-negative float), then exponent = rule(max of the ring); one thread
__device__ __forceinline__ void scale_state_push(ScaleState* st, uint32_t amax_bits, int target_exp)
{
    const int n = st->hist_len;
    st->amax_last = __uint_as_float(amax_bits);
    st->ring[st->pos] = __uint_as_float(amax_bits);
    st->pos = (st->pos + 1) % n;
    if (st->filled < n) st->filled++;
    uint32_t m = 0;
    for (int j = 0; j < st->filled; j++) m = max(m, __float_as_uint(st->ring[j]));  // non-negative floats order as integers
    st->scale_exp = scale_exp_from_amax(m, target_exp);
}

__device__ __forceinline__ int resolve_scale_exp(const ConvParams& p)
{
    if (p.d_amax_bits) return scale_exp_from_amax(*p.d_amax_bits, p.target_exp);
    if (p.d_scale_exp) return clamp_exp(*p.d_scale_exp);
    return p.scale_exp;
}

// amax contribution of a value: |x| for finite x, ignored (NaN) otherwise; fmaxf drops NaN operands
__device__ __forceinline__ float amax_step(float acc, float x) { return fmaxf(acc, fmaf(x, 0.0f, fabsf(x))); }

__device__ __forceinline__ void block_amax_commit(float acc, uint32_t* accum)
{
    __shared__ uint32_t s_part[kThreads / 32];
    uint32_t v = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(acc));  // non-negative floats order as integers
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        v = threadIdx.x < kThreads / 32 ? s_part[threadIdx.x] : 0u;
        v = __reduce_max_sync(0xFFFFFFFFu, v);
        if (threadIdx.x == 0 && v) atomicMax(accum, v);
    }
}

// launch with programmatic stream serialization (see pdl_* above)
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace
}  // namespace hif8
