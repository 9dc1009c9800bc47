/*
 * hif8.h -- C ABI of the B200 (sm_100a) HiFloat8 conversion library.
 *
 * HiFloat8 (HiF8) is the 8-bit tapered floating-point format of "Ascend HiFloat8 Format for Deep
 * Learning" (arXiv 2409.16626), Section 2.1: one byte = sign | dot field (prefix code, Table 2) |
 * sign-magnitude exponent with implicit leading 1 (Table 3) | 3/2/1-bit mantissa; normal values follow
 * Eq. 1, the denormal extension follows Eq. 2; 0x00 is the single zero, 0x80 is NaN, 0x6F / 0xEF are
 * +-Inf (Table 4).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller (any CUDA allocation); the library
 *     never allocates, frees or copies to the host, and never synchronises.  All work is enqueued on
 *     `stream` (a cudaStream_t; NULL = the legacy default stream) of the current device.
 *   - Tensors are contiguous, element count `n`.  Any byte alignment is accepted; 16-byte aligned
 *     pointers take the vectorised path, others a slower scalar kernel with identical results.
 *   - Return value: HIF8_OK or an error code (see hif8_status_string).  Argument errors are detected
 *     before anything is launched and leave all outputs untouched.  NaN / Inf inputs are data.
 *   - A conversion whose source and destination byte ranges intersect is rejected with HIF8_ERR_OVERLAP
 *     (host-side range test; the kernels read and write in an order that makes no promise for aliased data).
 *   - `scale_exp` is the exponent E of a power-of-two scale 2^E (Section 4.2: scale factors are
 *     integer powers of two, so scaling only adds to the exponent), limited to [-126, 126].
 *   - The library needs a CUDA device of compute capability 10.0 and fails with HIF8_ERR_CUDA elsewhere.
 */
#ifndef HIF8_H
#define HIF8_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* hif8_stream_t; /* same type as cudaStream_t */

/* element formats of the high-precision side (Section 3: FP32, FP16 and BF16 sources) */
typedef enum { HIF8_F32 = 0, HIF8_BF16 = 1, HIF8_F16 = 2 } hif8_dtype_t;

/* rounding methods of Section 3 */
typedef enum {
    HIF8_RND_TA = 0,  /* Section 3.1: round half away from zero (the default everywhere)               */
    HIF8_RND_HR = 1,  /* Eq. 3: hybrid -- TA if |E| < 4, simplified stochastic rounding if |E| >= 4    */
    HIF8_RND_SSR = 2, /* Section 3.2 simplified SR for every E: SR14 (FP32 source), SR2 (FP16 / BF16)  */
    HIF8_RND_TE = 3,  /* Section 3.1: round half to even                                               */
    HIF8_RND_SR = 4   /* Section 3.2 standard SR; thresholds from Philox4x32-10 keyed by `seed`         */
} hif8_round_t;

/* the two options of Section 3 */
enum {
    HIF8_FLAG_SATURATE = 1u,   /* overflow (and a source +-Inf) gives +-2^15 instead of +-Inf */
    HIF8_FLAG_NAN_TO_ZERO = 2u /* a source NaN gives 0x00 instead of 0x80                     */
};

enum {
    HIF8_OK = 0,
    HIF8_ERR_NULL = 1,        /* a required pointer is NULL                         */
    HIF8_ERR_DTYPE = 2,       /* unknown element format                             */
    HIF8_ERR_ROUND = 3,       /* unknown rounding method                            */
    HIF8_ERR_FLAGS = 4,       /* unknown option bits                                */
    HIF8_ERR_SCALE_RANGE = 5, /* scale or target exponent outside [-126, 126]       */
    HIF8_ERR_SHAPE = 6,       /* negative or unsupported extent / leading dimension */
    HIF8_ERR_ALIGN = 7,       /* GEMM operand not 16-byte aligned                   */
    HIF8_ERR_WORKSPACE = 8,   /* workspace missing or too small                     */
    HIF8_ERR_CUDA = 9,        /* a CUDA call failed (launch error, wrong device)    */
    HIF8_ERR_DEVICE_TIMEOUT = 10, /* a bounded device-side wait gave up            */
    HIF8_ERR_OVERLAP = 11     /* source and destination share bytes (Section 3: a conversion reads one tensor and
                                 writes another; only hif8_fake_quant may run in place, dst == src exactly)   */
};

/* which call a workspace size is asked for */
enum { HIF8_WS_AMAX_SCALE_ENCODE = 0, HIF8_WS_FAKE_QUANT = 1, HIF8_WS_GEMM = 2 };

/*
 * High-precision tensor -> HiF8 bytes (Section 3: rounding of FP32 / FP16 / BF16 data into the format).
 *   dst[i] = To_HiF8_<rnd>( src[i] * 2^scale_exp )
 * The scaled value is rounded as if 1.5*2^15 were representable; a result of that magnitude or more is
 * +-Inf (or +-2^15 with HIF8_FLAG_SATURATE).  Magnitudes that round to zero give 0x00 for either sign.
 * src: n elements of `src_dtype`; dst: n bytes; they must not overlap (HIF8_ERR_OVERLAP).  `seed` is used by HIF8_RND_SR only:
 * element i takes word (i mod 4) of Philox4x32-10 with counter (i/4, 0, 0) and key `seed`; its top 24 bits
 * (FP32 source) or 16 bits (16-bit sources) are the threshold T of Section 3.2.
 */
int hif8_encode(const void* src, int src_dtype, uint8_t* dst, size_t n, int scale_exp, int rnd,
                unsigned flags, uint64_t seed, hif8_stream_t stream);

/*
 * hif8_encode of a source that is generated instead of read: element i is the FP32 value whose encoding is
 * first_pattern + i (modulo 2^32), i = 0 .. n-1, n <= 2^32.  This is the exhaustive sweep over FP32 inputs (every
 * exponent including the denormal extension of Eq. 2, underflow to the single zero, overflow, Inf and NaN patterns of
 * Section 2.1 / Table 4) without a 4-byte-per-element source tensor: the call only writes, one byte per element.
 * HIF8_RND_SR draws the word of index i.  Arguments and errors otherwise as hif8_encode.
 */
int hif8_encode_f32_patterns(uint32_t first_pattern, uint8_t* dst, size_t n, int scale_exp, int rnd, unsigned flags,
                             uint64_t seed, hif8_stream_t stream);

/*
 * HiF8 bytes -> high-precision tensor (Eq. 1, Eq. 2, Table 4 specials), with the descale of
 * Algorithm 1 ("Restore"):   dst[i] = value(src[i]) * 2^(-scale_exp)
 * rounded to nearest-even into `dst_dtype` when not representable (only possible at the far ends of the
 * scale range, or for FP16 destinations).  0x80 gives the canonical quiet NaN, 0x6F / 0xEF give +-Inf.
 * src: n bytes; dst: n elements; no overlap (HIF8_ERR_OVERLAP).
 */
int hif8_decode(const uint8_t* src, void* dst, int dst_dtype, size_t n, int scale_exp,
                hif8_stream_t stream);

/*
 * Per-tensor scaled conversion (Section 5.1 "Per-Tensor Scaling"; Algorithm 1 "Scale & Cast").
 *   d_scale_exp_in == NULL  (just-in-time):  amax = max |src[i]| over finite elements;
 *        scale_exp = clamp(target_exp - floor(log2 amax), -126, 126)  (0 if amax is 0), so that
 *        amax * 2^scale_exp lies in [2^target_exp, 2^(target_exp+1)); then dst = To_HiF8(src * 2^scale_exp).
 *        Two kernels, the scale never leaves the device.
 *   d_scale_exp_in != NULL  (delayed scaling: Section 5.1 measures amax once per ten iterations): the scale exponent
 *        is read from that device int; amax of this tensor is still produced for the next update.  One pass.
 * Outputs (device scalars, each may be NULL): d_amax_out (float, exact), d_scale_exp_out (int, the exponent
 * used), d_scale_out (float 2^scale_exp).  workspace: hif8_workspace_bytes(HIF8_WS_AMAX_SCALE_ENCODE, n)
 * bytes of device memory, 256-byte aligned, contents irrelevant on entry and undefined on return.
 * target_exp in [-22, 15]; 14 keeps amax just below the largest finite value 2^15.
 */
int hif8_amax_scale_encode(const void* src, int src_dtype, uint8_t* dst, size_t n, int target_exp, int rnd,
                           unsigned flags, uint64_t seed, const int* d_scale_exp_in, float* d_amax_out,
                           int* d_scale_exp_out, float* d_scale_out, void* workspace,
                           size_t workspace_bytes, hif8_stream_t stream);

/*
 * Amax alone (Section 5.1, per-tensor scaling: the largest magnitude of each GEMM input tensor is measured at a fixed
 * cadence of iterations and the tensor's scale follows from it):
 *   *d_amax_out = max |src[i]| over the finite elements (0 if there is none), as an exact float.
 * One read of the tensor.  workspace as for hif8_amax_scale_encode.  The caller derives the next scale exponent
 * from it (or lets hif8_amax_scale_encode do both in one call).
 */
int hif8_amax(const void* src, int src_dtype, size_t n, float* d_amax_out, void* workspace, size_t workspace_bytes,
              hif8_stream_t stream);

/*
 * The second half of the just-in-time form on its own: the scale exponent is derived on the device from an amax the
 * caller already has in device memory, scale_exp = clamp(target_exp - floor(log2 *d_amax), -126, 126) (0 if it is 0),
 * then dst = To_HiF8_<rnd>(src * 2^scale_exp).  *d_amax must be a non-negative float.  Together with hif8_amax this
 * splits hif8_amax_scale_encode where a tensor is sharded over several GPUs: each rank reduces its shard, the ranks
 * combine the 4-byte values with a max all-reduce, and each converts its shard with the common exponent (Section 5.1:
 * one scale factor per GEMM input tensor).  Optional outputs as in hif8_amax_scale_encode.  No workspace.
 */
int hif8_encode_from_amax(const void* src, int src_dtype, uint8_t* dst, size_t n, int target_exp, int rnd, unsigned flags,
                          uint64_t seed, const float* d_amax, int* d_scale_exp_out, float* d_scale_out,
                          hif8_stream_t stream);

/*
 * hif8_amax_scale_encode without a caller-supplied workspace.  (The paper has no counterpart: this entry
 * point exists for the benefit of the calling environment only.)
 *
 * Who needs it: code that must not, or cannot, obtain device memory at the point of the call -- a plug-in that
 * runs inside another framework's memory pool and may not allocate behind its back, a call site inside a
 * real-time or fault-handling path where cudaMalloc's implicit synchronisation and possible failure are not
 * acceptable, or a process whose memory budget was handed out completely at start-up.  Such callers still pass
 * their input and output tensors; the few bytes of scratch the amax reduction needs come from a
 * HIF8_STATIC_SCRATCH_BYTES-byte array inside the library image, resident on every device that loads the
 * library until the process exits.
 *
 * Same arguments, results and errors as hif8_amax_scale_encode minus the workspace pair, plus:
 *   - n > HIF8_STATIC_MAX_ELEMENTS is rejected with HIF8_ERR_SHAPE before anything is launched.
 *   - No cudaMalloc / cudaFree / allocating library routine is called, now or later.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress); make that
 *     first call outside any stream capture.
 *   - All calls on a device share the one array.  Each call clears the words it needs on `stream` before
 *     using them, so back-to-back calls on one stream are safe; two calls that can overlap on the GPU
 *     (different streams, no dependency) race on it and give wrong scales -- serialise them, or use
 *     hif8_amax_scale_encode with separate workspaces.
 */
#define HIF8_STATIC_SCRATCH_BYTES 256
#define HIF8_STATIC_MAX_ELEMENTS ((size_t)1 << 32)
int hif8_amax_scale_encode_static(const void* src, int src_dtype, uint8_t* dst, size_t n, int target_exp, int rnd,
                                  unsigned flags, uint64_t seed, const int* d_scale_exp_in, float* d_amax_out,
                                  int* d_scale_exp_out, float* d_scale_out, hif8_stream_t stream);

/*
 * Per-channel scaled conversion of a weight matrix (Section 4.2 and the closing remarks of Section 5 and Section 6 name
 * the combination of one scale per activation tensor with one scale per weight channel).  W is [rows, cols] row-major and
 * contiguous; every output channel has its own power-of-two scale:
 *   channel_axis = 0: channel = row    (weights stored [N,K]);   channel_axis = 1: channel = column (stored [K,N]).
 *   d_scale_exp_in == NULL: per channel, amax over the channel's finite elements and
 *        scale_exp = clamp(target_exp - floor(log2 amax), -126, 126) (0 for an all-zero channel), the per-tensor rule
 *        of hif8_amax_scale_encode applied to the channel alone; d_amax [channels] receives the amax values (it is also
 *        the accumulator of the reduction and must not be NULL).
 *   d_scale_exp_in != NULL: the exponents are read from that device array [channels]; d_amax is not touched.
 *   dst[r, c] = To_HiF8_<rnd>( W[r, c] * 2^scale_exp[channel(r, c)] ), same layout as W, one byte per element.
 * d_scale_exp_out [channels] (may be NULL; may equal d_scale_exp_in): the exponents used, ready for
 * hif8_gemm_channel_scaled.  HIF8_RND_SR draws the word of flat index r * cols + c, as hif8_encode would.
 * Needs no workspace.  The fast path wants 16-byte aligned pointers and rows (cols * element size a multiple of 16);
 * anything else takes a slower element-wise path with identical results.
 */
int hif8_channel_amax_scale_encode(const void* W, int src_dtype, uint8_t* dst, int64_t rows, int64_t cols,
                                   int channel_axis, int target_exp, int rnd, unsigned flags, uint64_t seed,
                                   const int* d_scale_exp_in, float* d_amax, int* d_scale_exp_out,
                                   hif8_stream_t stream);

/*
 * The every-N-iterations cadence of per-tensor scaling in training (Section 5.1: scale factors start at 1; once per ten
 * iterations the amax of each tensor is measured and its scale updated; the scale in force is applied in every
 * iteration, updated or not).  The paper does not give the update rule; this library keeps, per tensor, the exponent
 * in force and a ring of the last `hist_len` measured amax values, and after a measurement sets
 *   scale_exp = clamp(target_exp - floor(log2 max(ring)), -126, 126)      (0 while every entry is 0)
 * which takes effect from the next conversion on.  The state lives in HIF8_SCALE_STATE_BYTES of device memory
 * (256-byte aligned) owned by the caller; nothing returns to the host.
 *   hif8_scale_state_init:      exponent 0, empty ring of hist_len entries (1..HIF8_SCALE_HISTORY_MAX).
 *   hif8_delayed_scale_encode:  dst = To_HiF8_<rnd>(src * 2^(exponent in force)) in one pass over src.  With
 *        measure != 0 (the caller's "iteration % N == 0") the same pass also reduces amax of src, and the last
 *        thread block to finish pushes it into the ring and updates the exponent (one kernel launch either way).  The first int of the state is the exponent
 *        in force (readable as the d_scale_exp_a / d_scale_exp_w of hif8_gemm), the float at byte 16 the last amax.
 */
#define HIF8_SCALE_STATE_BYTES 1024
#define HIF8_SCALE_HISTORY_MAX 32
int hif8_scale_state_init(void* d_state, int hist_len, hif8_stream_t stream);
int hif8_delayed_scale_encode(const void* src, int src_dtype, uint8_t* dst, size_t n, int rnd, unsigned flags,
                              uint64_t seed, void* d_state, int measure, int target_exp, hif8_stream_t stream);

/*
 * Adaptive loss scaling (Section 5.1, "Adaptive Loss-Scaling (ALS)"), resident on the device.
 * The loss scale is 2^scale_exp.  After each backward pass: hif8_check_finite over the (scaled) gradient tensors ORs
 * "holds an Inf or NaN" into *d_found_inf (a device int the caller zeroes once; hif8_als_update clears it again), then
 * hif8_als_update advances the controller:
 *   overflow          -> scale / 2, clean-iteration count = 0
 *   no overflow       -> count + 1; when it reaches the scale window -> scale * 2, count = 0
 *   scale window      : walks the list {1, 20, 50, 100, 200, 500, 1000}: three increases of the scale since the last
 *                       window change move it up one entry; three decreases not interrupted by an increase move it
 *                       down one entry; a window change clears both counts; it stops at the ends of the list.
 * The paper starts from scale 2^32 and window 20 (init_scale_exp = 32, init_window_index = 1).
 * State: HIF8_ALS_STATE_BYTES of device memory, 16-byte aligned, eight ints the caller may read at any time:
 *   [0] scale_exp  [1] window  [2] window index  [3] clean iterations  [4] increases counted  [5] decreases in a row
 *   [6] iterations seen  [7] iterations that overflowed.
 * The optimizer step of an overflowed iteration is the caller's to skip (it can test the flag on the device before
 * hif8_als_update clears it).  Nothing here returns to the host or synchronises.
 */
#define HIF8_ALS_STATE_BYTES 64
int hif8_als_state_init(void* d_state, int init_scale_exp, int init_window_index, hif8_stream_t stream);
int hif8_als_update(void* d_state, int* d_found_inf, hif8_stream_t stream);
/* *d_found_inf |= (some src[i] is +-Inf or NaN); one read of the tensor; src must be aligned to its element size */
int hif8_check_finite(const void* src, int dtype, size_t n, int* d_found_inf, hif8_stream_t stream);

/*
 * Quantize-dequantize in the source format (Section 4: the paper's experiments simulate the format by replacing every
 * value with its nearest HiF8-representable one):   dst[i] = value( To_HiF8_<rnd>(src[i] * 2^e) ) * 2^(-e)   in `dtype`.
 *   use_amax == 0: e = scale_or_target_exp.  No workspace needed (may be NULL).
 *   use_amax == 1: e derived from the tensor's amax with target exponent scale_or_target_exp, as in
 *                  hif8_amax_scale_encode (two kernels); workspace as for HIF8_WS_FAKE_QUANT.
 * dst may be the same pointer as src (in place); any other overlap is rejected with HIF8_ERR_OVERLAP.
 * d_amax_out / d_scale_exp_out: optional device scalars as above.
 */
int hif8_fake_quant(const void* src, void* dst, int dtype, size_t n, int use_amax, int scale_or_target_exp,
                    int rnd, unsigned flags, uint64_t seed, float* d_amax_out, int* d_scale_exp_out,
                    void* workspace, size_t workspace_bytes, hif8_stream_t stream);

/*
 * GEMM with HiF8 operands decoded in-kernel (Algorithm 1, "MatMul & Restore"; Section 4.1: only the GEMM
 * inputs are HiF8):   C[m,n] = 2^-(sa+sw) * sum_k value(Aq[m,k]) * value(Wq[k,n])
 * Decoded values are exact in BF16; products are accumulated in FP32 on the tensor cores.
 *   Aq: [M,K] row-major bytes, leading dimension lda.  Wq: [K,N] (w_is_nk = 0) or [N,K] (w_is_nk = 1)
 *   row-major bytes, leading dimension ldw.  C: [M,N] row-major, `c_dtype` HIF8_BF16 or HIF8_F32, ldc.
 *   d_scale_exp_a / d_scale_exp_w: device ints sa, sw (NULL = 0).
 * Pointers and leading dimensions (in bytes) must be multiples of 16 (HIF8_ERR_ALIGN); K must be a positive
 * multiple of 16 (HIF8_ERR_SHAPE).  NaN / Inf codes propagate as in IEEE arithmetic.
 * workspace: at least hif8_workspace_bytes(HIF8_WS_GEMM, 0) = 256 bytes, 16-byte aligned; its first int is a device
 * status word that the call clears and the kernel sets if one of its bounded waits ever gives up (see
 * hif8_gemm_status).  With only that, the fused kernel decodes the HiF8 byte tiles of every CTA pair inside the
 * tensor-core kernel (W into shared memory, an A given as [M,K] straight into tensor memory).
 * With hif8_workspace_bytes(HIF8_WS_GEMM, M*K + K*N) bytes, 256-byte aligned, and contiguous operands (lda = K,
 * ldw = row length of Wq), each operand byte is instead decoded once into the workspace (BF16, exact) and the
 * tensor-core kernel streams BF16 tiles: several times faster for compute-bound shapes, same results.
 * In between -- hif8_workspace_bytes(HIF8_WS_GEMM, M*K) bytes or more, 256-byte aligned, A contiguous -- A alone is
 * expanded into the workspace and the kernel decodes only the W tiles (any ldw): for when the weight's BF16 copy does
 * not fit but the activation's does; same results.  A workspace with room for both operands takes this form too while
 * the product is too small to win the pass over W back (see hif8_gemm_path_policy).
 * Products with at most 64 rows of A (and A given as [M,K]) take a weight-streaming kernel whatever the workspace;
 * with the workspace size above it spreads the weight bytes evenly over all SMs (partial sums of a column slab that
 * two SMs share go through the workspace and are added in a fixed order: results are reproducible run to run) and,
 * with A contiguous, first expands the few rows of A to BF16 there (one small launch more, same results).
 */
int hif8_gemm(const uint8_t* Aq, int64_t lda, const uint8_t* Wq, int64_t ldw, int w_is_nk, void* C,
              int64_t ldc, int c_dtype, int M, int N, int K, const int* d_scale_exp_a,
              const int* d_scale_exp_w, void* workspace, size_t workspace_bytes, hif8_stream_t stream);

/*
 * hif8_gemm with one weight exponent per output channel (per-tensor activation scale, per-channel weight scales):
 *   C[m,n] = 2^-(sa + sw[n]) * sum_k value(Aq[m,k]) * value(Wq[k,n]),   d_scale_exp_w_channel: device int [N], not NULL.
 * Everything else as hif8_gemm.
 */
int hif8_gemm_channel_scaled(const uint8_t* Aq, int64_t lda, const uint8_t* Wq, int64_t ldw, int w_is_nk, void* C,
                             int64_t ldc, int c_dtype, int M, int N, int K, const int* d_scale_exp_a,
                             const int* d_scale_exp_w_channel, void* workspace, size_t workspace_bytes,
                             hif8_stream_t stream);

/*
 * The general form of the HiF8 GEMM, covering the backward pass of Y = X W (Section 3: the activation gradient is
 * converted with TA or hybrid rounding; Section 4.1: activation, weight and activation gradient are the GEMM inputs):
 *   dgrad  dX[M,K'] = dY[M,N'] W^T :  Aq = dYq [M,N'],           Wq = the forward weight bytes [K',N'], w_is_nk = 1
 *   wgrad  dW[K',N'] = X^T dY      :  Aq = Xq [M',K'], a_is_km = 1 (A is read as [K,M] = [M',K']), Wq = dYq [M',N'], w_is_nk = 0
 * so neither backward GEMM needs a transposed copy of a byte tensor.
 *   C[m,n] (+)= 2^-(sa + sw_n) * sum_k value(A(m,k)) * value(W(k,n))
 *   a_is_km = 0: Aq is [M,K] row-major (lda >= K);  a_is_km = 1: Aq is [K,M] row-major (lda >= M).
 *   w_is_nk as in hif8_gemm.  sw_n = d_scale_exp_w_channel[n] if that pointer is given, else *d_scale_exp_w (or 0).
 *   accumulate != 0: the product is added to the existing contents of C (FP32 C: one rounding per element per call;
 *   BF16 C: sum formed in FP32, then rounded to nearest even) -- gradient accumulation over micro-batches.
 * Alignment, K, workspace and status conventions as in hif8_gemm (the decode-once path needs contiguous operands).
 */
int hif8_gemm_ex(const uint8_t* Aq, int64_t lda, int a_is_km, const uint8_t* Wq, int64_t ldw, int w_is_nk, void* C,
                 int64_t ldc, int c_dtype, int M, int N, int K, const int* d_scale_exp_a, const int* d_scale_exp_w,
                 const int* d_scale_exp_w_channel, int accumulate, void* workspace, size_t workspace_bytes,
                 hif8_stream_t stream);

/*
 * Conversion with transposed store: dst[c, r] = To_HiF8_<rnd>( src[r, c] * 2^e ), src [rows, cols] row-major of
 * `src_dtype`, dst [cols, rows] bytes.  For frameworks that keep a second, transposed byte copy of a GEMM operand
 * (the backward GEMMs contract over the other dimension); hif8_gemm_ex does not need it.
 *   e = *d_scale_exp if that device pointer is given (delayed scaling), else scale_exp.
 *   HIF8_RND_SR draws the word of the SOURCE flat index r * cols + c, so the codes equal those of hif8_encode, moved.
 * The fast path wants 16-byte aligned pointers, cols a multiple of the 16-byte vector (4 FP32 / 8 16-bit elements) and
 * rows a multiple of 16; anything else takes an element-wise path with identical results.
 */
int hif8_encode_transpose(const void* src, int src_dtype, uint8_t* dst, int64_t rows, int64_t cols, int scale_exp,
                          const int* d_scale_exp, int rnd, unsigned flags, uint64_t seed, hif8_stream_t stream);

/*
 * Host-side query of the status word of a finished hif8_gemm: copies it from `workspace`, SYNCHRONISES `stream`,
 * and returns HIF8_OK or HIF8_ERR_DEVICE_TIMEOUT (the output tile of the CTA that gave up is then undefined).
 * The only entry point that blocks the host.
 */
int hif8_gemm_status(const void* workspace, hif8_stream_t stream);

/*
 * Which general kernel a large workspace selects.  HIF8_GEMM_PATH_AUTO (the default): with room for both operands W is
 * expanded too only when the product is large enough to win that pass back (from about 1500 rows of A with [K,N] weights,
 * about 4800 with [N,K] weights); below that A alone is expanded.  HIF8_GEMM_PATH_EXPAND_BOTH: both operands are expanded whenever the workspace has room (for
 * measurements and tests of that kernel on small products).  Process-wide; returns the previous setting (0 or 1), or
 * HIF8_ERR_FLAGS for an unknown one.  Results do not depend on it.
 */
enum { HIF8_GEMM_PATH_AUTO = 0, HIF8_GEMM_PATH_EXPAND_BOTH = 1 };
int hif8_gemm_path_policy(int policy);

/*
 * Status of the most recent GEMM-class call (hif8_gemm, hif8_gemm_ex, hif8_gemm_channel_scaled, hif8_pts_search,
 * hif8_selftest_wait_timeout) enqueued on `stream` of the current device, without the caller naming the workspace:
 * the library remembers, per stream, where that call's status word lives.  SYNCHRONISES `stream`, then returns HIF8_OK,
 * HIF8_ERR_DEVICE_TIMEOUT, or HIF8_ERR_CUDA (read failed, or another device is current).  HIF8_OK when no such call was
 * made on the stream.  The workspace of that call must still be allocated.  (Algorithm 1 has no counterpart; this is
 * the host-side end of the bounded device-side waits.)
 */
int hif8_last_device_status(hif8_stream_t stream);

/*
 * Self-test of the host-side caches (no device needed): the once-per-device set-up record and the tensor-map cache are
 * driven with synthetic keys; returns HIF8_OK, or HIF8_ERR_SHAPE with the number of the failed check in *failed_check.
 */
int hif8_selftest_host_caches(int* failed_check);

/*
 * Self-test of the device-side failure detection: launches one warp that waits, with a limit of `limit_ms`
 * milliseconds (1..1000), on a barrier that is never completed.  The wait gives up, the kernel records the status
 * word in `workspace` (first int, cleared by the call) and ends normally; hif8_gemm_status(workspace, stream) then
 * returns HIF8_ERR_DEVICE_TIMEOUT and the device stays usable.  No fault, trap or unbounded loop is involved.
 */
int hif8_selftest_wait_timeout(void* workspace, unsigned limit_ms, hif8_stream_t stream);

/*
 * Per-layer search of Algorithm 1 ("HiF8 Calibration with Per-Tensor Scaling"): for every (Ea, Ew) with both
 * exponents in [e_min, e_max] (the paper searches [-4, 5]):
 *     A_q = To_HiF8_TA(A * 2^Ea), W_q = To_HiF8_TA(W * 2^Ew);  O_q = (A_q x W_q) * 2^-(Ea+Ew);
 *     d_err[(Ea - e_min) * n + (Ew - e_min)] = MSE(O_q, O_ref) over all M*N outputs      (n = e_max - e_min + 1 <= 16)
 * and d_best[0], d_best[1] = the (Ea, Ew) of the smallest error (first one in that order on exact ties).
 * A: [M,K] row-major; W: [K,N] (w_is_nk = 0) or [N,K]; both contiguous, of `dtype`; O_ref: the layer's high-precision
 * output [M,N] as float, leading dimension ldo.  K and the row length of W must be multiples of 16.
 * All device memory; 2n encodes, n*n GEMMs with FP32 output and n*n reductions are enqueued on `stream`, nothing
 * returns to the host.  workspace: hif8_pts_workspace_bytes(M, N, K, n) bytes, 256-byte aligned; its first int is a
 * device status word as for hif8_gemm (hif8_pts_status reads it, synchronising the stream).
 */
int hif8_pts_search(const void* A, const void* W, int dtype, int w_is_nk, const float* O_ref, int64_t ldo, int M, int N,
                    int K, int e_min, int e_max, float* d_err, int* d_best, void* workspace, size_t workspace_bytes,
                    hif8_stream_t stream);
size_t hif8_pts_workspace_bytes(int M, int N, int K, int n_exp);
int hif8_pts_status(const void* workspace, hif8_stream_t stream);

/* bytes of device workspace a call needs (which = HIF8_WS_*; n = element count; for HIF8_WS_GEMM: 0 for the
 * minimum, or M*K + K*N for the decode-once path) */
size_t hif8_workspace_bytes(int which, size_t n);

/* static, NUL-terminated description of a status code */
const char* hif8_status_string(int status);

/*
 * Number of kernels the library has launched from this process since it was loaded (all entry points,
 * all streams).  Host-side counter for tests and benchmarks.
 */
uint64_t hif8_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* HIF8_H */
