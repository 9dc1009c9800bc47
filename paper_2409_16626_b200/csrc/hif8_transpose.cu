// Conversion with transposed store: dst[c, r] = To_HiF8(src[r, c] * 2^e).  (Backward-pass operand form: the GEMMs of
// the backward pass contract over the other dimension of the activation / gradient tensors.)
//
// A block converts a tile of 128 source rows by 8 source vectors (32 FP32 or 64 16-bit columns).  Thread (rq, cv)
// loads the four vectors of rows 4 rq .. 4 rq + 3 in vector-column cv (four independent 16-byte loads; a warp covers
// four full 128-byte lines per instruction), converts them, and packs the four bytes of each of its columns into one
// 32-bit word of a shared tile held transposed ([column][row / 4], 16-byte chunks XOR-swizzled by the column's vector
// index: conflict-free both ways).  The block then writes each column of the tile as 128 contiguous bytes of a dst row.
// Traffic is that of the flat encoder: one read of the source, one byte written per element.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "hif8.h"
#include "hif8_device.cuh"
#include "hif8_internal.cuh"

namespace hif8 {
extern std::atomic<uint64_t> g_launches;
namespace {

struct TrParams {
    const void* src;
    uint8_t* dst;
    long long rows, cols;
    int scale_exp;
    const int* d_scale_exp;
    unsigned flags;
    unsigned long long seed;
    int rows_on_x;  // grid x counts row tiles (only for more than 65535 row tiles); else x counts column strips
};

constexpr int kTileRows = 128;
constexpr int kTileVecs = 8;          // vector-columns per tile
constexpr int kTileWords = kTileRows / 4;  // words per tile column (128 code bytes)

// Grid: x = tile of 128 source rows, y = strip of 8 source vectors (looped when there are more strips than the grid's
// y extent).  Blocks with consecutive x write adjacent 128-byte segments of the same dst rows.
template <int SRC, int MODE>
__global__ void __launch_bounds__(kThreads, MODE == HIF8_RND_SR ? 4 : 6) encode_transpose_kernel(const TrParams p)
{
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    constexpr int TC = kTileVecs * PV;  // source columns per tile
    __shared__ SmemTables sm;
    // tile[c][w]: code bytes of source column c, rows 4w .. 4w+3 in word w; the 16-byte chunk index (w / 4) is XORed
    // with the column's vector index so that both the word stores below and the 16-byte reads are conflict-free
    __shared__ __align__(16) uint32_t tile[TC * kTileWords];
    constexpr bool kSum16 = SRC == HIF8_BF16 && (MODE == HIF8_RND_HR || MODE == HIF8_RND_SSR);  // packed BF16 arithmetic
    if (kSum16) setup_sum16<MODE>(sm.ta, sm.thr, p.flags);
    else setup_tables<true, MODE != HIF8_RND_TA, false, MODE, SRC>(sm, p.flags);
    const float scale = pow2f(p.d_scale_exp ? clamp_exp(*p.d_scale_exp) : p.scale_exp);
    const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
    const long long nvc = p.cols / PV;                        // vectors per source row
    const long long strips = (nvc + kTileVecs - 1) / kTileVecs;
    const int cv = threadIdx.x % kTileVecs, rq = threadIdx.x / kTileVecs;
    // x = strip of source columns (fastest), y = tile of source rows: blocks that run together read neighbouring
    // 128-byte pieces of the same source rows, i.e. whole lines of the row-major source
    const unsigned bx = p.rows_on_x ? blockIdx.x : blockIdx.y, by = p.rows_on_x ? blockIdx.y : blockIdx.x;
    const unsigned gy = p.rows_on_x ? gridDim.y : gridDim.x;
    const long long r0 = (long long)bx * kTileRows;
    const bool rows_full = r0 + kTileRows <= p.rows;
    uint32_t* const my_words = tile + cv * PV * kTileWords + (((rq >> 2) ^ cv) << 2) + (rq & 3);

    for (long long tc = by; tc < strips; tc += gy) {
        const long long v0 = tc * kTileVecs, vcol = v0 + cv;
        const bool full = rows_full && v0 + kTileVecs <= nvc;
        const uint4* sp = reinterpret_cast<const uint4*>(p.src) + (r0 + rq * 4) * nvc + vcol;
        uint4 v[4];
        if (full) {
#pragma unroll
            for (int j = 0; j < 4; j++) v[j] = __ldcs(sp + j * nvc);
        } else {
#pragma unroll
            for (int j = 0; j < 4; j++)
                v[j] = (r0 + rq * 4 + j < p.rows && vcol < nvc) ? __ldcs(sp + j * nvc) : make_uint4(0, 0, 0, 0);
        }
        if (MODE == HIF8_RND_SR) {
            // one generator call serves a whole source vector: rows outermost, the words of all columns accumulate
            uint32_t packed[PV];
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const unsigned long long u = (unsigned long long)(r0 + rq * 4 + j) * nvc + vcol;  // flat vector index in the source
                uint4 q0 = philox4x32_10((uint32_t)(u * (PV / 4)), (uint32_t)((u * (PV / 4)) >> 32), k0, k1), q1 = q0;
                if (PV == 8) q1 = philox4x32_10((uint32_t)(u * 2 + 1), (uint32_t)((u * 2 + 1) >> 32), k0, k1);
                const uint32_t rw[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
                for (int k = 0; k < PV; k++) {
                    float x; uint32_t raw;
                    unpack<SRC>(v[j], k, x, raw);
                    const uint32_t c = encode_one<MODE, SRC>(x, raw, scale, sm.ta, sm.thr, rw[k]) << (8 * j);
                    packed[k] = j ? (packed[k] | c) : c;
                }
            }
#pragma unroll
            for (int k = 0; k < PV; k++) my_words[k * kTileWords] = packed[k];
        } else if constexpr (kSum16) {
            // a source word holds two neighbouring columns: the codes of four rows are gathered into one word per column
            const uint32_t ns2 = neg_scale_bf16x2(scale);
#pragma unroll
            for (int m = 0; m < 4; m++) {
                uint32_t c[4], y[4];
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    const uint32_t w = m == 0 ? v[j].x : (m == 1 ? v[j].y : (m == 2 ? v[j].z : v[j].w));
                    y[j] = mul_bf16x2(w, ns2);
                    c[j] = encode_sum16(w, y[j], sm.ta, sm.thr);
                }
                const uint32_t c01 = __byte_perm(c[0], c[1], 0x5140), c23 = __byte_perm(c[2], c[3], 0x5140);
                const uint32_t s01 = __byte_perm(y[0], y[1], 0x7351), s23 = __byte_perm(y[2], y[3], 0x7351);
                // a set (inverted) sign clears bit 7
                my_words[(2 * m) * kTileWords] = __byte_perm(c01, c23, 0x5410) & (~__byte_perm(s01, s23, 0x5410) | 0x7F7F7F7Fu);
                my_words[(2 * m + 1) * kTileWords] = __byte_perm(c01, c23, 0x7632) & (~__byte_perm(s01, s23, 0x7632) | 0x7F7F7F7Fu);
            }
        } else if constexpr (MODE == HIF8_RND_TA) {
            // The table is read sign-free (see ta_magnitude_code: the byte lookups share the load/store pipe with the
            // tile) and the signs of the four rows of a column go back onto the packed word: bit 7 of every code that
            // is not the single zero (code + 0x7F carries into bit 7 for 0x01 .. 0x80; NaN, 0x80, keeps its encoding).
#pragma unroll
            for (int k = 0; k < PV; k++) {
                uint32_t c[4], w[4];
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    float x; uint32_t raw;
                    unpack<SRC>(v[j], k, x, raw);
                    c[j] = ta_magnitude_code(x, scale, sm.ta);
                    constexpr int kDiv = SRC == HIF8_F32 ? 1 : 2;
                    w[j] = (k / kDiv) == 0 ? v[j].x : ((k / kDiv) == 1 ? v[j].y : ((k / kDiv) == 2 ? v[j].z : v[j].w));
                }
                const bool top = SRC == HIF8_F32 || (k & 1);  // the element's sign is bit 7 of byte 3 (else of byte 1) of its word
                const uint32_t s01 = __byte_perm(w[0], w[1], top ? 0x0073u : 0x0051u), s23 = __byte_perm(w[2], w[3], top ? 0x0073u : 0x0051u);
                const uint32_t word = c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24);
                my_words[k * kTileWords] = word | ((word + 0x7F7F7F7Fu) & __byte_perm(s01, s23, 0x5410u) & 0x80808080u);
            }
        } else {
            // columns outermost: the four codes of a column are packed and stored at once
#pragma unroll
            for (int k = 0; k < PV; k++) {
                uint32_t c[4];
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    float x; uint32_t raw;
                    unpack<SRC>(v[j], k, x, raw);
                    c[j] = encode_one<MODE, SRC>(x, raw, scale, sm.ta, sm.thr, 0u);
                }
                my_words[k * kTileWords] = c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24);
            }
        }
        __syncthreads();
        // column c of the tile = 128 bytes of dst row (v0 * PV + c), starting at byte r0; 16 bytes per thread
        constexpr int kSegs = kTileRows / 16;
        const int seg = threadIdx.x % kSegs, c_lo = threadIdx.x / kSegs;
        uint8_t* dp = p.dst + (v0 * PV + c_lo) * p.rows + r0 + seg * 16;
#pragma unroll
        for (int i = 0; i < TC * kSegs / kThreads; i++) {
            const int c = c_lo + i * (kThreads / kSegs);
            const uint4 q = *reinterpret_cast<const uint4*>(tile + c * kTileWords + ((seg ^ ((c / PV) & 7)) << 2));
            // rows is a multiple of 16 on this path: a segment is all in or all out
            if (full || (v0 * PV + c < p.cols && r0 + seg * 16 < p.rows)) __stcs(reinterpret_cast<uint4*>(dp + (long long)i * (kThreads / kSegs) * p.rows), q);
        }
        if (tc + gy < strips) __syncthreads();  // (block-uniform) the tile is read out before the next one is stored
    }
}

// any shape and alignment: one thread per source element
template <int SRC, int MODE>
__global__ void __launch_bounds__(kThreads) encode_transpose_scalar_kernel(const TrParams p)
{
    __shared__ SmemTables sm;
    setup_tables<true, MODE != HIF8_RND_TA, false, MODE, SRC>(sm, p.flags);
    const float scale = pow2f(p.d_scale_exp ? clamp_exp(*p.d_scale_exp) : p.scale_exp);
    const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
    const unsigned long long n = (unsigned long long)p.rows * (unsigned long long)p.cols;
    for (unsigned long long i = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += (unsigned long long)gridDim.x * kThreads) {
        const unsigned long long r = i / (unsigned long long)p.cols, c = i - r * (unsigned long long)p.cols;
        float x; uint32_t raw;
        load_scalar<SRC>(p.src, i, x, raw);
        uint32_t word = 0;
        if (MODE == HIF8_RND_SR) {
            const uint4 q = philox4x32_10((uint32_t)(i >> 2), (uint32_t)(i >> 34), k0, k1);
            word = philox_word(q, (unsigned)i & 3u);
        }
        p.dst[c * (unsigned long long)p.rows + r] = (uint8_t)encode_one<MODE, SRC>(x, raw, scale, sm.ta, sm.thr, word);
    }
}

// HiF8 bytes [rows, cols] -> BF16 [cols, rows] (exact).  Used by the GEMM's decode-once path for an A operand given as
// [K, M]: the tensor-core kernel then always streams a K-major A.  A block stages a 64 x 256 byte tile in shared memory
// (rows padded by one word: a column walk then touches successive banks), then eight lanes write the 64 values of one
// output row segment as 128 contiguous bytes.
constexpr int kDtRows = 64, kDtCols = 256, kDtStride = kDtCols + 4;

__global__ void __launch_bounds__(kThreads) decode_transpose_bf16_kernel(const uint8_t* __restrict__ src, unsigned short* __restrict__ dst,
                                                                         long long rows, long long cols)
{
    __shared__ uint32_t tile[kDtRows * kDtStride / 4];
    __shared__ unsigned short lut[256];
    lut[threadIdx.x] = (unsigned short)(decode_bits_f32(threadIdx.x) >> 16);  // every HiF8 value is exact in BF16
    const long long tiles_c = (cols + kDtCols - 1) / kDtCols, tiles_r = (rows + kDtRows - 1) / kDtRows;
    const uint8_t* tb = reinterpret_cast<const uint8_t*>(tile);
    for (long long tix = blockIdx.x; tix < tiles_c * tiles_r; tix += gridDim.x) {
        const long long tc = tix / tiles_r, tr = tix % tiles_r;
        const long long r0 = tr * kDtRows, c0 = tc * kDtCols;
        __syncthreads();  // the previous tile has been read out (and the table is complete)
        // 64 rows x 16 chunks of 16 bytes
#pragma unroll
        for (int i = 0; i < kDtRows * (kDtCols / 16) / kThreads; i++) {
            const int v = i * kThreads + threadIdx.x, r = v / (kDtCols / 16), ch = v % (kDtCols / 16);
            uint4 q = make_uint4(0, 0, 0, 0);
            if (r0 + r < rows && c0 + ch * 16 < cols) q = __ldcs(reinterpret_cast<const uint4*>(src + (r0 + r) * cols + c0 + ch * 16));
            uint32_t* d = tile + (r * kDtStride + ch * 16) / 4;
            d[0] = q.x; d[1] = q.y; d[2] = q.z; d[3] = q.w;
        }
        __syncthreads();
        // output row c (a source column), eight source rows per lane: 16 bytes of BF16
#pragma unroll
        for (int i = 0; i < kDtCols * (kDtRows / 8) / kThreads; i++) {
            const int v = i * kThreads + threadIdx.x, c = v / (kDtRows / 8), seg = v % (kDtRows / 8);
            if (c0 + c >= cols || r0 + seg * 8 >= rows) continue;  // rows is a multiple of 8: a segment is all in or all out
            uint32_t h[8];
#pragma unroll
            for (int k = 0; k < 8; k++) h[k] = lut[tb[(seg * 8 + k) * kDtStride + c]];
            __stcs(reinterpret_cast<uint4*>(dst + (c0 + c) * rows + r0 + seg * 8),
                   make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16)));
        }
    }
}

template <int SRC, int MODE>
int launch(const TrParams& p, bool vec, int sms, cudaStream_t st)
{
    if (vec) {
        constexpr int PV = SrcTraits<SRC>::kPerVec;
        const long long nvc = p.cols / PV;
        const long long strips = (nvc + kTileVecs - 1) / kTileVecs, row_tiles = (p.rows + kTileRows - 1) / kTileRows;
        if (row_tiles > 0x7FFFFFFFll) return HIF8_ERR_SHAPE;
        // up to four strips per block (two under round half away, whose set-up is light: 35.2 against 36.5 us on BF16
        // 8192 x 8192, where hybrid rounding measured 47.5 against 45.5 us) while at least one full wave of resident
        // blocks remains: the per-block table set-up is then shared by several tiles
        const long long wave = (long long)sms * 6;
        const long long cap = MODE == HIF8_RND_TA ? 2 : 4;
        long long per_block = row_tiles * strips / wave;
        per_block = per_block < 1 ? 1 : per_block > cap ? cap : per_block;
        long long gy = (strips + per_block - 1) / per_block;
        if (gy > 65535) gy = 65535;
        TrParams q = p;
        q.rows_on_x = row_tiles > 65535 ? 1 : 0;
        const dim3 grid = q.rows_on_x ? dim3((unsigned)row_tiles, (unsigned)gy) : dim3((unsigned)gy, (unsigned)row_tiles);
        encode_transpose_kernel<SRC, MODE><<<grid, kThreads, 0, st>>>(q);
    } else {
        const unsigned long long n = (unsigned long long)p.rows * (unsigned long long)p.cols;
        const unsigned long long need = (n + kThreads - 1) / kThreads, cap = (unsigned long long)sms * 32;
        encode_transpose_scalar_kernel<SRC, MODE><<<(unsigned)(need < cap ? need : cap), kThreads, 0, st>>>(p);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

template <int SRC>
int launch_mode(int rnd, const TrParams& p, bool vec, int sms, cudaStream_t st)
{
    switch (rnd) {
        case HIF8_RND_TA: return launch<SRC, HIF8_RND_TA>(p, vec, sms, st);
        case HIF8_RND_HR: return launch<SRC, HIF8_RND_HR>(p, vec, sms, st);
        case HIF8_RND_SSR: return launch<SRC, HIF8_RND_SSR>(p, vec, sms, st);
        case HIF8_RND_TE: return launch<SRC, HIF8_RND_TE>(p, vec, sms, st);
        default: return launch<SRC, HIF8_RND_SR>(p, vec, sms, st);
    }
}

}  // namespace

int decode_transpose_bf16(const uint8_t* src, void* dst, long long rows, long long cols, cudaStream_t st)
{
    if (rows <= 0 || cols <= 0 || (rows & 7) || (cols & 15)) return HIF8_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(src) & 15u) || (reinterpret_cast<uintptr_t>(dst) & 15u)) return HIF8_ERR_ALIGN;
    const long long tiles = ((cols + kDtCols - 1) / kDtCols) * ((rows + kDtRows - 1) / kDtRows);
    decode_transpose_bf16_kernel<<<(unsigned)(tiles < 0x7FFFFFFFll ? tiles : 0x7FFFFFFFll), kThreads, 0, st>>>(
        src, reinterpret_cast<unsigned short*>(dst), rows, cols);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

}  // namespace hif8

using namespace hif8;

extern "C" int hif8_encode_transpose(const void* src, int src_dtype, uint8_t* dst, int64_t rows, int64_t cols, int scale_exp,
                                     const int* d_scale_exp, int rnd, unsigned flags, uint64_t seed, hif8_stream_t stream)
{
    if (src_dtype != HIF8_F32 && src_dtype != HIF8_BF16 && src_dtype != HIF8_F16) return HIF8_ERR_DTYPE;
    if (rnd < HIF8_RND_TA || rnd > HIF8_RND_SR) return HIF8_ERR_ROUND;
    if (flags & ~(unsigned)(HIF8_FLAG_SATURATE | HIF8_FLAG_NAN_TO_ZERO)) return HIF8_ERR_FLAGS;
    if (scale_exp < -126 || scale_exp > 126) return HIF8_ERR_SCALE_RANGE;
    if (rows < 0 || cols < 0) return HIF8_ERR_SHAPE;
    if (rows == 0 || cols == 0) return HIF8_OK;
    if (!src || !dst) return HIF8_ERR_NULL;
    if (ranges_overlap(src, (size_t)rows * (size_t)cols * dtype_bytes(src_dtype), dst, (size_t)rows * (size_t)cols))
        return HIF8_ERR_OVERLAP;
    int sms; int rc = checked_device(&sms);
    if (rc) return rc;
    const int pv = src_dtype == HIF8_F32 ? 4 : 8;
    const bool vec = !(reinterpret_cast<uintptr_t>(src) & 15u) && !(reinterpret_cast<uintptr_t>(dst) & 15u) && cols % pv == 0 &&
                     rows % 16 == 0;
    TrParams p{};
    p.src = src; p.dst = dst; p.rows = rows; p.cols = cols; p.scale_exp = scale_exp; p.d_scale_exp = d_scale_exp;
    p.flags = flags; p.seed = seed;
    cudaStream_t st = (cudaStream_t)stream;
    switch (src_dtype) {
        case HIF8_F32: return launch_mode<HIF8_F32>(rnd, p, vec, sms, st);
        case HIF8_BF16: return launch_mode<HIF8_BF16>(rnd, p, vec, sms, st);
        default: return launch_mode<HIF8_F16>(rnd, p, vec, sms, st);
    }
}
