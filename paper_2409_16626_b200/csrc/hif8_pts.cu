// Per-layer search of Algorithm 1 ("HiF8 Calibration with Per-Tensor Scaling"): for every pair of power-of-two
// scale exponents (Ea, Ew) of a grid, cast activation and weight to HiF8 with round-half-away, multiply, restore, and
// measure the mean squared error against the layer's high-precision output; keep the pair with the smallest error.
//
// Built from the library's own entry points: each operand is encoded once per exponent (hif8_encode), each pair is one
// hif8_gemm (FP32 output, descale by the device-resident exponents), followed by a squared-error reduction in double
// precision; a last one-block kernel turns the sums into the MSE table and takes the argmin.  Nothing returns to the
// host in between.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "hif8.h"

namespace hif8 {
extern std::atomic<uint64_t> g_launches;
namespace {

constexpr int kMaxExps = 16;
constexpr size_t kCtlBytes = 4096;  // [0]: status, [64..): int exps[16], [256..): double sums[256]

struct PtsCtl {
    int status;
    int pad[15];
    int exps[kMaxExps];
    int pad2[32];
    double sums[kMaxExps * kMaxExps];
};
static_assert(sizeof(PtsCtl) <= kCtlBytes, "control block too large");

__global__ void pts_init_kernel(PtsCtl* ctl, int e_min, int n_exp)
{
    const int i = threadIdx.x;
    if (i == 0) ctl->status = 0;
    if (i < n_exp) ctl->exps[i] = e_min + i;
    if (i < kMaxExps * kMaxExps) ctl->sums[i] = 0.0;
}

// sums[slot] += sum over the tile of (C - O)^2; also latches a GEMM device status into ctl->status
__global__ void __launch_bounds__(256) pts_sqerr_kernel(const float* __restrict__ C, const float* __restrict__ O, long long ldo,
                                                        int M, int N, PtsCtl* ctl, int slot, const int* gemm_status)
{
    double acc = 0.0;
    const long long total = (long long)M * N;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long m = i / N, n = i - m * N;
        const double d = (double)C[i] - (double)O[m * ldo + n];
        acc += d * d;
    }
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    __shared__ double s_part[8];
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; w++) t += s_part[w];
        atomicAdd(&ctl->sums[slot], t);
        if (blockIdx.x == 0 && *gemm_status) atomicCAS(&ctl->status, 0, *gemm_status);
    }
}

__global__ void pts_finish_kernel(const PtsCtl* ctl, int e_min, int n_exp, double inv_count, float* d_err, int* d_best)
{
    if (threadIdx.x != 0) return;
    int best = 0;
    double best_v = ctl->sums[0];
    for (int i = 0; i < n_exp * n_exp; i++) {
        const double v = ctl->sums[i];
        d_err[i] = (float)(v * inv_count);
        if (v < best_v) { best_v = v; best = i; }  // first minimum in row-major (Ea, Ew) order
    }
    d_best[0] = e_min + best / n_exp;
    d_best[1] = e_min + best % n_exp;
}

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace
}  // namespace hif8

using namespace hif8;

extern "C" size_t hif8_pts_workspace_bytes(int M, int N, int K, int n_exp)
{
    if (M <= 0 || N <= 0 || K <= 0 || n_exp <= 0 || n_exp > kMaxExps) return 0;
    const size_t mk = (size_t)M * K, kn = (size_t)K * N;
    return kCtlBytes + align256(mk) * n_exp + align256(kn) * n_exp + align256((size_t)M * N * 4) +
           align256(hif8_workspace_bytes(HIF8_WS_GEMM, mk + kn));
}

extern "C" int hif8_pts_search(const void* A, const void* W, int dtype, int w_is_nk, const float* O_ref, int64_t ldo, int M,
                               int N, int K, int e_min, int e_max, float* d_err, int* d_best, void* workspace,
                               size_t workspace_bytes, hif8_stream_t stream)
{
    if (dtype != HIF8_F32 && dtype != HIF8_BF16 && dtype != HIF8_F16) return HIF8_ERR_DTYPE;
    const int n_exp = e_max - e_min + 1;
    if (n_exp < 1 || n_exp > kMaxExps || e_min < -126 || e_max > 126) return HIF8_ERR_SCALE_RANGE;
    if (M <= 0 || N <= 0 || K <= 0 || (K & 15) || ((w_is_nk ? K : N) & 15) || ldo < N) return HIF8_ERR_SHAPE;
    if (!A || !W || !O_ref || !d_err || !d_best) return HIF8_ERR_NULL;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < hif8_pts_workspace_bytes(M, N, K, n_exp))
        return HIF8_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t mk = (size_t)M * K, kn = (size_t)K * N;
    unsigned char* base = reinterpret_cast<unsigned char*>(workspace);
    PtsCtl* ctl = reinterpret_cast<PtsCtl*>(base);
    unsigned char* aq = base + kCtlBytes;
    unsigned char* wq = aq + align256(mk) * n_exp;
    float* C = reinterpret_cast<float*>(wq + align256(kn) * n_exp);
    unsigned char* gws = reinterpret_cast<unsigned char*>(C) + align256((size_t)M * N * 4);
    const size_t gws_bytes = hif8_workspace_bytes(HIF8_WS_GEMM, mk + kn);

    pts_init_kernel<<<1, 256, 0, st>>>(ctl, e_min, n_exp);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) return HIF8_ERR_CUDA;
    for (int i = 0; i < n_exp; i++) {  // "Scale & Cast", once per exponent and operand
        int rc = hif8_encode(A, dtype, aq + align256(mk) * i, mk, e_min + i, HIF8_RND_TA, 0, 0, stream);
        if (rc == HIF8_OK) rc = hif8_encode(W, dtype, wq + align256(kn) * i, kn, e_min + i, HIF8_RND_TA, 0, 0, stream);
        if (rc != HIF8_OK) return rc;
    }
    const long long total = (long long)M * N;
    const unsigned grid = (unsigned)(total / 1024 + 1 < 1184 ? total / 1024 + 1 : 1184);
    for (int ia = 0; ia < n_exp; ia++)
        for (int iw = 0; iw < n_exp; iw++) {  // "MatMul & Restore", "Quantization Error"
            int rc = hif8_gemm(aq + align256(mk) * ia, K, wq + align256(kn) * iw, w_is_nk ? K : N, w_is_nk, C, N, HIF8_F32, M, N, K,
                               &ctl->exps[ia], &ctl->exps[iw], gws, gws_bytes, stream);
            if (rc != HIF8_OK) return rc;
            pts_sqerr_kernel<<<grid, 256, 0, st>>>(C, O_ref, ldo, M, N, ctl, ia * n_exp + iw, reinterpret_cast<const int*>(gws));
            g_launches.fetch_add(1, std::memory_order_relaxed);
        }
    pts_finish_kernel<<<1, 32, 0, st>>>(ctl, e_min, n_exp, 1.0 / ((double)M * (double)N), d_err, d_best);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

extern "C" int hif8_pts_status(const void* workspace, hif8_stream_t stream)
{
    return hif8_gemm_status(workspace, stream);  // same convention: first int of the workspace
}
