// Declarations shared between the translation units of the library (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace hif8 {

struct GemmParams {
    void* C;
    long long ldc;
    int c_is_f32;
    int M, N, K;
    const int* d_sa;
    const int* d_sw;
    int accumulate;           // nonzero: C += result instead of C = result
    const int* d_sw_channel;  // when set: one weight exponent per output column [N]; d_sw is then ignored
    int* status;
    int tiles_m, tiles_n;
    // when err_sum is set the epilogue stores nothing: it adds sum (result - err_ref)^2 of its tile to *err_sum
    const float* err_ref;
    long long ld_ref;
    double* err_sum;
    // batch_n = n > 0: n x n products in one launch, A variant ia with W variant iw for product ia * n + iw; d_sa / d_sw
    // are then arrays of n exponents and err_sum an array of n * n sums
    int batch_n;
    int c_by_tma;             // fused kernel: the BF16 result tile is staged in shared memory and written by tile stores
};

// C (or the squared error) from operands that are already BF16 in device memory: a_bf [M,K], w_bf [K,N] or (w_is_nk) [N,K],
// both contiguous.  Fills in the tile counts of `p`; p.status must point at a zeroed device int.
// In a batch the variants of an operand are `*_stack_stride` elements apart (multiples of 8).
int launch_bf16_pair_gemm(const void* a_bf, const void* w_bf, int w_is_nk, GemmParams p, cudaStream_t st,
                          long long a_stack_stride = 0, long long w_stack_stride = 0);

// dst[c][r] = BF16 value of the HiF8 byte src[r][c]; src [rows, cols] contiguous (rows a multiple of 8, cols of 16), both
// pointers 16-byte aligned
int decode_transpose_bf16(const uint8_t* src, void* dst, long long rows, long long cols, cudaStream_t st);

// Remembers `word` (a device int that a kernel sets when one of its bounded waits gives up) as the status word of the
// latest GEMM-class call on stream `st` of the current device; hif8_last_device_status reads it back.
void note_status_word(cudaStream_t st, const int* word);

// True when the byte ranges [a, a + a_bytes) and [b, b + b_bytes) share at least one byte (empty ranges share none).
inline bool ranges_overlap(const void* a, size_t a_bytes, const void* b, size_t b_bytes)
{
    const uintptr_t pa = reinterpret_cast<uintptr_t>(a), pb = reinterpret_cast<uintptr_t>(b);
    return a_bytes && b_bytes && pa < pb + b_bytes && pb < pa + a_bytes;
}
inline size_t dtype_bytes(int dtype) { return dtype == 0 ? 4 : 2; }  // HIF8_F32 : HIF8_BF16 / HIF8_F16

// SM count of the current device; HIF8_ERR_CUDA unless it is a compute-capability-10.0 device
int checked_device(int* sms);

}  // namespace hif8
