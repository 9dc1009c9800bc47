// Per-channel scaled conversion of weight matrices (Section 5.1: per-tensor scaling for activations, per-channel
// scaling for weights).  W is [rows, cols] row-major; a channel is a row (weights stored [N,K]) or a column ([K,N]).
//
// Channel = row: a group of threads per row.  A row of up to 32 KiB is read once into registers, reduced over the
// group (no atomics) to its amax, and converted from the registers while the next row's loads are in flight; longer
// rows are read twice, the second time from L1/L2.
// Channel = column: two kernels over the same tiling, a strip of up to 256 vector-columns (4 KiB of a row) by
// `rows_per_block` rows per block.  A warp reads 512 contiguous bytes of one row per instruction; each lane keeps the
// running maxima (first kernel) or the scales (second kernel) of its own 4 or 8 columns in registers while it walks
// down the rows.  Warps stacked over the same columns combine their maxima in shared memory, so a block issues one
// atomicMax per column.
// The amax array holds bit patterns of non-negative floats (they order as unsigned integers), so it is both the
// accumulator and the result the caller reads as float.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "hif8.h"
#include "hif8_device.cuh"
#include "hif8_internal.cuh"

namespace hif8 {
extern std::atomic<uint64_t> g_launches;
namespace {

struct ChanParams {
    const void* src;
    uint8_t* dst;
    long long rows, cols;
    const int* d_se_in;   // exponents given by the caller, one per channel, or null
    uint32_t* amax_bits;  // per-channel amax (bit patterns); used when d_se_in is null
    int* d_se_out;        // may be null
    int target_exp;
    unsigned flags;
    unsigned long long seed;
};

__device__ __forceinline__ int channel_exp(const ChanParams& p, long long ch)
{
    return p.d_se_in ? clamp_exp(p.d_se_in[ch]) : scale_exp_from_amax(p.amax_bits[ch], p.target_exp);
}

// bytes of one converted source vector -> global memory
template <int PV> __device__ __forceinline__ void store_codes(uint8_t* dst, unsigned long long vec_index, const uint32_t (&codes)[PV])
{
    const uint32_t w0 = codes[0] | (codes[1] << 8) | (codes[2] << 16) | (codes[3] << 24);
    if (PV == 4) __stcs(reinterpret_cast<uint32_t*>(dst) + vec_index, w0);
    else {
        const uint32_t w1 = codes[4] | (codes[5] << 8) | (codes[6] << 16) | (codes[7] << 24);
        __stcs(reinterpret_cast<uint2*>(dst) + vec_index, make_uint2(w0, w1));
    }
}

// the stochastic words of the PV elements of flat vector u (element i takes word i % 4 of counter i / 4)
template <int MODE, int PV> __device__ __forceinline__ void sr_words(unsigned long long u, uint32_t k0, uint32_t k1, uint32_t (&rw)[8])
{
    uint4 r0 = make_uint4(0, 0, 0, 0), r1 = r0;
    if (MODE == HIF8_RND_SR) {
        r0 = philox4x32_10((uint32_t)(u * (PV / 4)), (uint32_t)((u * (PV / 4)) >> 32), k0, k1);
        if (PV == 8) r1 = philox4x32_10((uint32_t)(u * 2 + 1), (uint32_t)((u * 2 + 1) >> 32), k0, k1);
    }
    rw[0] = r0.x; rw[1] = r0.y; rw[2] = r0.z; rw[3] = r0.w; rw[4] = r1.x; rw[5] = r1.y; rw[6] = r1.z; rw[7] = r1.w;
}

// ------------------------------------------------------------------------------------------------
// channel = row
// ------------------------------------------------------------------------------------------------
constexpr int kRowCache = 8;  // vectors per thread a row may occupy to be held in registers: 32 KiB per row

// maximum of non-negative bit patterns over the group of `gs` threads (a power of two, 32 .. kThreads, aligned in the
// block) that shares a row; every thread of the group gets the result.  Called by all threads of the block.
__device__ __forceinline__ uint32_t group_max(uint32_t v, uint32_t* s_part, int gs)
{
    v = __reduce_max_sync(0xFFFFFFFFu, v);
    if (gs == 32) return v;
    __syncthreads();  // the previous use of s_part is over
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = v;
    __syncthreads();
    const int w0 = (threadIdx.x / gs) * (gs / 32);
    v = 0;
    for (int w = 0; w < gs / 32; w++) v = max(v, s_part[w0 + w]);
    return v;
}

// Rows that fit in registers (at most NV vectors per thread of a group of gs threads).  A block works through
// `iters` consecutive sets of kThreads / gs rows; the loads of the next set are issued before the current one is
// reduced and converted, so every row is read exactly once and the memory latency is covered by the arithmetic of the
// previous row.  Short rows get small groups so that a thread still holds about four vectors.
template <int SRC, int MODE, int NV>
__global__ void __launch_bounds__(kThreads, 4) row_channel_kernel(const ChanParams p, int gs, int iters)
{
    __shared__ SmemTables sm;
    __shared__ uint32_t s_part[kThreads / 32];
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    setup_tables<true, MODE != HIF8_RND_TA, false, MODE, SRC>(sm, p.flags);
    const unsigned long long nv = (unsigned long long)p.cols / PV;  // vectors per row (cols is a multiple of PV here)
    const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
    const int groups = kThreads / gs, g = threadIdx.x / gs, t = threadIdx.x % gs;
    const uint4* base = reinterpret_cast<const uint4*>(p.src);
    const long long first = (long long)blockIdx.x * iters * groups + g;

    // NV <= kUnroll: two register sets, the next row is in flight while this one is processed; larger rows use one set
    constexpr bool kPrefetch = NV <= kUnroll;
    uint4 cur[NV], nxt[kPrefetch ? NV : 1];
    if (kPrefetch) {
#pragma unroll
        for (int j = 0; j < NV; j++) {
            const unsigned long long u = (unsigned long long)j * gs + t;
            nxt[j] = (first < p.rows && u < nv) ? __ldcs(base + (unsigned long long)first * nv + u) : make_uint4(0, 0, 0, 0);
        }
    }
    for (int it = 0; it < iters; it++) {
        const long long row = first + (long long)it * groups, row_next = row + groups;
        const bool live = row < p.rows;  // a group past the last row only takes part in the barriers
        if (kPrefetch) {
#pragma unroll
            for (int j = 0; j < NV; j++) cur[j] = nxt[j];
            if (it + 1 < iters) {
#pragma unroll
                for (int j = 0; j < NV; j++) {
                    const unsigned long long u = (unsigned long long)j * gs + t;
                    nxt[j] = (row_next < p.rows && u < nv) ? __ldcs(base + (unsigned long long)row_next * nv + u) : make_uint4(0, 0, 0, 0);
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < NV; j++) {
                const unsigned long long u = (unsigned long long)j * gs + t;
                cur[j] = (live && u < nv) ? __ldcs(base + (unsigned long long)row * nv + u) : make_uint4(0, 0, 0, 0);
            }
        }
        int se = 0;
        if (p.d_se_in) se = live ? clamp_exp(p.d_se_in[row]) : 0;
        else {
            float m = 0.f;
#pragma unroll
            for (int j = 0; j < NV; j++)
#pragma unroll
                for (int k = 0; k < PV; k++) {
                    float x; uint32_t raw;
                    unpack<SRC>(cur[j], k, x, raw);
                    m = amax_step(m, x);
                }
            const uint32_t b = group_max(__float_as_uint(m), s_part, gs);
            if (t == 0 && live) p.amax_bits[row] = b;
            se = scale_exp_from_amax(b, p.target_exp);
        }
        if (t == 0 && live && p.d_se_out) p.d_se_out[row] = se;
        const float scale = pow2f(se);
        if (live) {
#pragma unroll
            for (int j = 0; j < NV; j++) {
                const unsigned long long u = (unsigned long long)j * gs + t;
                if (u >= nv) continue;
                const unsigned long long flat = (unsigned long long)row * nv + u;
                uint32_t rw[8], codes[PV];
                sr_words<MODE, PV>(flat, k0, k1, rw);
#pragma unroll
                for (int k = 0; k < PV; k++) {
                    float x; uint32_t raw;
                    unpack<SRC>(cur[j], k, x, raw);
                    codes[k] = encode_one<MODE, SRC>(x, raw, scale, sm.ta, sm.thr, rw[k]);
                }
                store_codes<PV>(p.dst, flat, codes);
            }
        }
    }
}

// Longer rows: one block per row, read twice; the second read is served by L1/L2.
template <int SRC, int MODE>
__global__ void __launch_bounds__(kThreads) long_row_channel_kernel(const ChanParams p)
{
    __shared__ SmemTables sm;
    __shared__ uint32_t s_part[kThreads / 32];
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    setup_tables<true, MODE != HIF8_RND_TA, false, MODE, SRC>(sm, p.flags);
    const unsigned long long nv = (unsigned long long)p.cols / PV;
    const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);

    for (long long row = blockIdx.x; row < p.rows; row += gridDim.x) {
        const uint4* src = reinterpret_cast<const uint4*>(p.src) + (unsigned long long)row * nv;
        int se;
        if (p.d_se_in) se = clamp_exp(p.d_se_in[row]);
        else {
            float m = 0.f;
            for (unsigned long long base = 0; base < nv; base += (unsigned long long)kThreads * kUnroll) {
                uint4 v[kUnroll];
#pragma unroll
                for (int j = 0; j < kUnroll; j++) {
                    const unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
                    v[j] = u < nv ? src[u] : make_uint4(0, 0, 0, 0);  // default caching: the second read wants these lines
                }
#pragma unroll
                for (int j = 0; j < kUnroll; j++)
#pragma unroll
                    for (int k = 0; k < PV; k++) {
                        float x; uint32_t raw;
                        unpack<SRC>(v[j], k, x, raw);
                        m = amax_step(m, x);
                    }
            }
            const uint32_t b = group_max(__float_as_uint(m), s_part, kThreads);
            if (threadIdx.x == 0) p.amax_bits[row] = b;
            se = scale_exp_from_amax(b, p.target_exp);
        }
        if (threadIdx.x == 0 && p.d_se_out) p.d_se_out[row] = se;
        const float scale = pow2f(se);
        for (unsigned long long base = 0; base < nv; base += (unsigned long long)kThreads * kUnroll) {
            uint4 v[kUnroll];
#pragma unroll
            for (int j = 0; j < kUnroll; j++) {
                const unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
                v[j] = u < nv ? __ldcs(src + u) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int j = 0; j < kUnroll; j++) {
                const unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
                if (u >= nv) continue;
                const unsigned long long flat = (unsigned long long)row * nv + u;
                uint32_t rw[8], codes[PV];
                sr_words<MODE, PV>(flat, k0, k1, rw);
#pragma unroll
                for (int k = 0; k < PV; k++) {
                    float x; uint32_t raw;
                    unpack<SRC>(v[j], k, x, raw);
                    codes[k] = encode_one<MODE, SRC>(x, raw, scale, sm.ta, sm.thr, rw[k]);
                }
                store_codes<PV>(p.dst, flat, codes);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// channel = column
// ------------------------------------------------------------------------------------------------
// A block is wx warps across (wx * 32 vector-columns: wx * 512 contiguous bytes of a row) by 8 / wx warps down.
// grid.x: strips of wx * 32 vector-columns; grid.y: groups of rows_per_block rows.  Wide strips keep the DRAM
// accesses of a block in long contiguous runs; narrow ones give small matrices enough blocks.
template <int SRC>
__global__ void __launch_bounds__(kThreads) col_amax_kernel(const ChanParams p, int rows_per_block, int wx)
{
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    __shared__ uint32_t s_max[kThreads / 32][32 * PV];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wy = (kThreads / 32) / wx, wxi = warp % wx, wyi = warp / wx;
    const long long nvc = p.cols / PV;
    const long long cv = ((long long)blockIdx.x * wx + wxi) * 32 + lane;
    const long long r0 = (long long)blockIdx.y * rows_per_block, r1 = min(r0 + rows_per_block, p.rows);
    float m[PV];
#pragma unroll
    for (int k = 0; k < PV; k++) m[k] = 0.f;
    if (cv < nvc) {
        const uint4* src = reinterpret_cast<const uint4*>(p.src) + cv;
        for (long long r = r0 + wyi; r < r1; r += wy * kUnroll) {
            uint4 v[kUnroll];
#pragma unroll
            for (int j = 0; j < kUnroll; j++) {
                const long long rr = r + wy * j;
                v[j] = rr < r1 ? __ldcs(src + rr * nvc) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int j = 0; j < kUnroll; j++)
#pragma unroll
                for (int k = 0; k < PV; k++) {
                    float x; uint32_t raw;
                    unpack<SRC>(v[j], k, x, raw);
                    m[k] = amax_step(m[k], x);
                }
        }
    }
#pragma unroll
    for (int k = 0; k < PV; k++) s_max[warp][lane * PV + k] = __float_as_uint(m[k]);
    __syncthreads();
    for (int idx = threadIdx.x; idx < wx * 32 * PV; idx += kThreads) {  // one atomic per column of the strip
        const int sx = idx / (32 * PV), within = idx % (32 * PV);
        uint32_t b = 0;
        for (int y = 0; y < wy; y++) b = max(b, s_max[y * wx + sx][within]);
        const long long col = ((long long)blockIdx.x * wx + sx) * 32 * PV + within;
        if (b && col < p.cols) atomicMax(p.amax_bits + col, b);
    }
}

template <int SRC, int MODE>
__global__ void __launch_bounds__(kThreads) col_encode_kernel(const ChanParams p, int rows_per_block, int wx)
{
    __shared__ SmemTables sm;
    constexpr int PV = SrcTraits<SRC>::kPerVec;
    setup_tables<true, MODE != HIF8_RND_TA, false, MODE, SRC>(sm, p.flags);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wy = (kThreads / 32) / wx, wxi = warp % wx, wyi = warp / wx;
    const long long nvc = p.cols / PV;
    const long long cv = ((long long)blockIdx.x * wx + wxi) * 32 + lane;
    if (cv >= nvc) return;
    const long long r0 = (long long)blockIdx.y * rows_per_block, r1 = min(r0 + rows_per_block, p.rows);
    const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
    float scale[PV];
#pragma unroll
    for (int k = 0; k < PV; k++) {
        const int se = channel_exp(p, cv * PV + k);
        scale[k] = pow2f(se);
        if (blockIdx.y == 0 && wyi == 0 && p.d_se_out) p.d_se_out[cv * PV + k] = se;
    }
    const uint4* src = reinterpret_cast<const uint4*>(p.src) + cv;
    for (long long r = r0 + wyi; r < r1; r += wy * kUnroll) {
        uint4 v[kUnroll];
#pragma unroll
        for (int j = 0; j < kUnroll; j++) {
            const long long rr = r + wy * j;
            v[j] = rr < r1 ? __ldcs(src + rr * nvc) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < kUnroll; j++) {
            const long long rr = r + wy * j;
            if (rr >= r1) continue;
            const unsigned long long flat = (unsigned long long)rr * nvc + cv;
            uint32_t rw[8], codes[PV];
            sr_words<MODE, PV>(flat, k0, k1, rw);
#pragma unroll
            for (int k = 0; k < PV; k++) {
                float x; uint32_t raw;
                unpack<SRC>(v[j], k, x, raw);
                codes[k] = encode_one<MODE, SRC>(x, raw, scale[k], sm.ta, sm.thr, rw[k]);
            }
            store_codes<PV>(p.dst, flat, codes);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// element-wise path: any alignment, any cols.  amax: one thread per (channel, slice of the channel).
// ------------------------------------------------------------------------------------------------
template <int SRC>
__global__ void __launch_bounds__(kThreads) chan_amax_scalar_kernel(const ChanParams p, int axis, int slices)
{
    const long long channels = axis == 0 ? p.rows : p.cols, len = axis == 0 ? p.cols : p.rows;
    const long long t = (long long)blockIdx.x * kThreads + threadIdx.x;
    // axis 1: neighbouring threads take neighbouring columns (coalesced); axis 0: a thread walks along its row slice
    const long long ch = t % channels, slice = t / channels;
    if (slice >= slices) return;
    const long long per = (len + slices - 1) / slices, j0 = slice * per, j1 = min(j0 + per, len);
    float m = 0.f;
    for (long long j = j0; j < j1; j++) {
        float x; uint32_t raw;
        load_scalar<SRC>(p.src, (unsigned long long)(axis == 0 ? ch * p.cols + j : j * p.cols + ch), x, raw);
        m = amax_step(m, x);
    }
    if (m > 0.f) atomicMax(p.amax_bits + ch, __float_as_uint(m));
}

template <int SRC, int MODE>
__global__ void __launch_bounds__(kThreads) chan_encode_scalar_kernel(const ChanParams p, int axis)
{
    __shared__ SmemTables sm;
    setup_tables<true, MODE != HIF8_RND_TA, false, MODE, SRC>(sm, p.flags);
    const unsigned long long n = (unsigned long long)p.rows * (unsigned long long)p.cols;
    const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
    for (unsigned long long i = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += (unsigned long long)gridDim.x * kThreads) {
        const long long r = (long long)(i / (unsigned long long)p.cols), c = (long long)(i - (unsigned long long)r * p.cols);
        const long long ch = axis == 0 ? r : c;
        const int se = channel_exp(p, ch);
        if (p.d_se_out && (axis == 0 ? c == 0 : r == 0)) p.d_se_out[ch] = se;
        float x; uint32_t raw;
        load_scalar<SRC>(p.src, i, x, raw);
        uint32_t word = 0;
        if (MODE == HIF8_RND_SR) {
            const uint4 q = philox4x32_10((uint32_t)(i >> 2), (uint32_t)(i >> 34), k0, k1);
            word = philox_word(q, (unsigned)i & 3u);
        }
        p.dst[i] = (uint8_t)encode_one<MODE, SRC>(x, raw, pow2f(se), sm.ta, sm.thr, word);
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct Plan {
    bool vec;  // 16-byte path
    int axis;
    int sms;
    int wx;  // warps across in the column kernels
    int rpb_encode, rpb_amax;  // rows per block
    dim3 grid_encode, grid_amax;
};

template <int SRC, int MODE>
int launch_encode(const ChanParams& p, const Plan& pl, cudaStream_t st)
{
    if (!pl.vec) {
        const unsigned long long n = (unsigned long long)p.rows * (unsigned long long)p.cols;
        unsigned long long need = (n + kThreads - 1) / kThreads, cap = (unsigned long long)pl.sms * 32;
        chan_encode_scalar_kernel<SRC, MODE><<<(unsigned)(need < cap ? need : cap), kThreads, 0, st>>>(p, pl.axis);
    } else if (pl.axis == 0) {
        const long long nv = p.cols / SrcTraits<SRC>::kPerVec;
        if (nv > (long long)kRowCache * kThreads) {
            const unsigned grid = (unsigned)(p.rows < 0x7FFFFFFFll ? p.rows : 0x7FFFFFFFll);
            long_row_channel_kernel<SRC, MODE><<<grid, kThreads, 0, st>>>(p);
        } else {
            // group size for about four vectors per thread; up to eight sets of rows per block while every SM still
            // gets eight blocks
            int gs = kThreads;
            while (gs > 32 && nv <= (long long)(gs / 2) * kUnroll) gs >>= 1;
            const long long sets = (p.rows + kThreads / gs - 1) / (kThreads / gs);
            int iters = nv <= (long long)kUnroll * gs ? 8 : 1;
            while (iters > 1 && (sets + iters - 1) / iters < (long long)pl.sms * 8) iters >>= 1;
            const long long blocks = (sets + iters - 1) / iters;
            if (blocks > 0x7FFFFFFFll) return HIF8_ERR_SHAPE;
            if (nv <= (long long)kUnroll * gs) row_channel_kernel<SRC, MODE, kUnroll><<<(unsigned)blocks, kThreads, 0, st>>>(p, gs, iters);
            else row_channel_kernel<SRC, MODE, kRowCache><<<(unsigned)blocks, kThreads, 0, st>>>(p, gs, iters);
        }
    } else {
        col_encode_kernel<SRC, MODE><<<pl.grid_encode, kThreads, 0, st>>>(p, pl.rpb_encode, pl.wx);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

template <int SRC>
int launch_mode(int rnd, const ChanParams& p, const Plan& pl, cudaStream_t st)
{
    switch (rnd) {
        case HIF8_RND_TA: return launch_encode<SRC, HIF8_RND_TA>(p, pl, st);
        case HIF8_RND_HR: return launch_encode<SRC, HIF8_RND_HR>(p, pl, st);
        case HIF8_RND_SSR: return launch_encode<SRC, HIF8_RND_SSR>(p, pl, st);
        case HIF8_RND_TE: return launch_encode<SRC, HIF8_RND_TE>(p, pl, st);
        default: return launch_encode<SRC, HIF8_RND_SR>(p, pl, st);
    }
}

template <int SRC>
int launch_amax(const ChanParams& p, const Plan& pl, cudaStream_t st)
{
    if (pl.vec && pl.axis == 0) return HIF8_OK;  // the row kernel reduces its own amax
    if (pl.vec) col_amax_kernel<SRC><<<pl.grid_amax, kThreads, 0, st>>>(p, pl.rpb_amax, pl.wx);
    else {
        const long long channels = pl.axis == 0 ? p.rows : p.cols, len = pl.axis == 0 ? p.cols : p.rows;
        // enough (channel, slice) threads to fill the device, slices of at least 64 elements
        long long slices = ((long long)pl.sms * 2048 + channels - 1) / channels;
        const long long max_slices = (len + 63) / 64;
        if (slices > max_slices) slices = max_slices;
        if (slices < 1) slices = 1;
        const long long threads = channels * slices;
        chan_amax_scalar_kernel<SRC><<<(unsigned)((threads + kThreads - 1) / kThreads), kThreads, 0, st>>>(p, pl.axis, (int)slices);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

}  // namespace
}  // namespace hif8

using namespace hif8;

extern "C" int hif8_channel_amax_scale_encode(const void* W, int src_dtype, uint8_t* dst, int64_t rows, int64_t cols,
                                              int channel_axis, int target_exp, int rnd, unsigned flags, uint64_t seed,
                                              const int* d_scale_exp_in, float* d_amax, int* d_scale_exp_out,
                                              hif8_stream_t stream)
{
    if (src_dtype != HIF8_F32 && src_dtype != HIF8_BF16 && src_dtype != HIF8_F16) return HIF8_ERR_DTYPE;
    if (rnd < HIF8_RND_TA || rnd > HIF8_RND_SR) return HIF8_ERR_ROUND;
    if (flags & ~(unsigned)(HIF8_FLAG_SATURATE | HIF8_FLAG_NAN_TO_ZERO)) return HIF8_ERR_FLAGS;
    if (target_exp < -22 || target_exp > 15) return HIF8_ERR_SCALE_RANGE;
    if (rows < 0 || cols < 0 || (channel_axis != 0 && channel_axis != 1)) return HIF8_ERR_SHAPE;
    const long long channels = channel_axis == 0 ? rows : cols;
    if (channels > 0x7FFFFFFFll * 64) return HIF8_ERR_SHAPE;
    if (rows == 0 || cols == 0) {
        // no element: every channel has amax 0 and exponent 0
        if (channels && !d_scale_exp_in) {
            if (!d_amax) return HIF8_ERR_NULL;
            if (cudaMemsetAsync(d_amax, 0, sizeof(float) * (size_t)channels, (cudaStream_t)stream) != cudaSuccess) return HIF8_ERR_CUDA;
            if (d_scale_exp_out &&
                cudaMemsetAsync(d_scale_exp_out, 0, sizeof(int) * (size_t)channels, (cudaStream_t)stream) != cudaSuccess)
                return HIF8_ERR_CUDA;
        }
        return HIF8_OK;
    }
    if (!W || !dst || (!d_scale_exp_in && !d_amax)) return HIF8_ERR_NULL;
    if (ranges_overlap(W, (size_t)rows * (size_t)cols * dtype_bytes(src_dtype), dst, (size_t)rows * (size_t)cols))
        return HIF8_ERR_OVERLAP;
    Plan pl{};
    int rc = checked_device(&pl.sms);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const int pv = src_dtype == HIF8_F32 ? 4 : 8;
    pl.axis = channel_axis;
    pl.vec = (reinterpret_cast<uintptr_t>(W) & 15u) == 0 && (reinterpret_cast<uintptr_t>(dst) & (size_t)(pv - 1)) == 0 &&
             cols % pv == 0;
    if (pl.vec && channel_axis == 1) {
        // Measured on 8192 x 28672 BF16: the conversion is fastest when a thread walks 32 rows, whatever the strip
        // width; the reduction when it walks about 128.  Strips of four warps (2 KiB of a row) unless the matrix is
        // narrower; fewer rows per thread while the grid would not give every SM eight blocks.
        const long long nvc = cols / pv;
        int wx = 4, rpt = 32;
        while (wx > 1 && nvc <= 32 * (wx / 2)) wx >>= 1;
        const long long strips = (nvc + 32 * wx - 1) / (32 * wx);
        const int wy = 8 / wx;
        while (rpt > 4 && strips * ((rows + rpt * wy - 1) / (rpt * wy)) < (long long)pl.sms * 8) rpt >>= 1;
        int rpt_a = 4 * rpt;  // the reduction likes longer walks, as long as every SM still gets eight blocks
        while (rpt_a > rpt && strips * ((rows + rpt_a * wy - 1) / (rpt_a * wy)) < (long long)pl.sms * 8) rpt_a >>= 1;
        const int rpb_e = rpt * wy, rpb_a = rpt_a * wy;
        const long long gy_e = (rows + rpb_e - 1) / rpb_e, gy_a = (rows + rpb_a - 1) / rpb_a;
        if (strips > 0x7FFFFFFFll || gy_e > 65535) pl.vec = false;  // outside the launch limits: element-wise path
        pl.wx = wx; pl.rpb_encode = rpb_e; pl.rpb_amax = rpb_a;
        pl.grid_encode = dim3((unsigned)strips, (unsigned)gy_e);
        pl.grid_amax = dim3((unsigned)strips, (unsigned)gy_a);
    }
    ChanParams p{};
    p.src = W; p.dst = dst; p.rows = rows; p.cols = cols; p.d_se_in = d_scale_exp_in;
    p.amax_bits = reinterpret_cast<uint32_t*>(d_amax); p.d_se_out = d_scale_exp_out;
    p.target_exp = target_exp; p.flags = flags; p.seed = seed;
    if (!d_scale_exp_in) {
        if (!(pl.vec && channel_axis == 0) &&
            cudaMemsetAsync(d_amax, 0, sizeof(float) * (size_t)channels, st) != cudaSuccess)
            return HIF8_ERR_CUDA;
        switch (src_dtype) {
            case HIF8_F32: rc = launch_amax<HIF8_F32>(p, pl, st); break;
            case HIF8_BF16: rc = launch_amax<HIF8_BF16>(p, pl, st); break;
            default: rc = launch_amax<HIF8_F16>(p, pl, st); break;
        }
        if (rc) return rc;
    }
    switch (src_dtype) {
        case HIF8_F32: return launch_mode<HIF8_F32>(rnd, p, pl, st);
        case HIF8_BF16: return launch_mode<HIF8_BF16>(rnd, p, pl, st);
        default: return launch_mode<HIF8_F16>(rnd, p, pl, st);
    }
}
