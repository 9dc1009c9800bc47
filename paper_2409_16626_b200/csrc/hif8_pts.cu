// Per-layer search of Algorithm 1 ("HiF8 Calibration with Per-Tensor Scaling"): for every pair of power-of-two
// scale exponents (Ea, Ew) of a grid, cast activation and weight to HiF8 with round-half-away, multiply, restore, and
// measure the mean squared error against the layer's high-precision output; keep the pair with the smallest error.
//
// Each operand is cast once per exponent (hif8_encode into a scratch byte buffer) and expanded once to BF16
// (hif8_decode, exact), so the n*n multiplications read ready BF16 operands.  All pairs are one launch of the
// tensor-core kernel (their tiles form one list for the persistent CTA pairs), whose epilogue restores the scale (2^-(Ea+Ew), device-resident exponents) and, instead of storing
// the product, adds the squared differences to the layer's output into one double per pair; a last one-block kernel
// turns the sums into the MSE table and takes the argmin.  Nothing returns to the host in between.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "hif8.h"
#include "hif8_internal.cuh"

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
    // control block, one scratch byte tensor, n BF16 copies of each operand
    return kCtlBytes + align256(mk > kn ? mk : kn) + (align256(mk * 2) + align256(kn * 2)) * (size_t)n_exp;
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
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return HIF8_ERR_CUDA;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (major != 10) return HIF8_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t mk = (size_t)M * K, kn = (size_t)K * N;
    unsigned char* base = reinterpret_cast<unsigned char*>(workspace);
    PtsCtl* ctl = reinterpret_cast<PtsCtl*>(base);
    unsigned char* q_tmp = base + kCtlBytes;
    unsigned char* a_bf = q_tmp + align256(mk > kn ? mk : kn);
    unsigned char* w_bf = a_bf + align256(mk * 2) * n_exp;

    pts_init_kernel<<<1, 256, 0, st>>>(ctl, e_min, n_exp);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) return HIF8_ERR_CUDA;
    for (int i = 0; i < n_exp; i++) {  // "Scale & Cast", once per exponent and operand; the HiF8 values as BF16
        int rc = hif8_encode(A, dtype, q_tmp, mk, e_min + i, HIF8_RND_TA, 0, 0, stream);
        if (rc == HIF8_OK) rc = hif8_decode(q_tmp, a_bf + align256(mk * 2) * i, HIF8_BF16, mk, 0, stream);
        if (rc == HIF8_OK) rc = hif8_encode(W, dtype, q_tmp, kn, e_min + i, HIF8_RND_TA, 0, 0, stream);
        if (rc == HIF8_OK) rc = hif8_decode(q_tmp, w_bf + align256(kn * 2) * i, HIF8_BF16, kn, 0, stream);
        if (rc != HIF8_OK) return rc;
    }
    GemmParams p{};
    p.M = M; p.N = N; p.K = K;
    p.status = &ctl->status;
    note_status_word((cudaStream_t)stream, &ctl->status);
    p.err_ref = O_ref; p.ld_ref = ldo;
    // "MatMul & Restore" and "Quantization Error" of all n * n pairs in one launch: the tiles of every product form one
    // list that the persistent CTA pairs walk through, so only the very last wave of the whole search is ragged
    p.d_sa = ctl->exps; p.d_sw = ctl->exps;
    p.err_sum = ctl->sums;
    p.batch_n = n_exp;
    {
        const int rc = launch_bf16_pair_gemm(a_bf, w_bf, w_is_nk, p, st, (long long)(align256(mk * 2) / 2), (long long)(align256(kn * 2) / 2));
        if (rc != HIF8_OK) return rc;
    }
    pts_finish_kernel<<<1, 32, 0, st>>>(ctl, e_min, n_exp, 1.0 / ((double)M * (double)N), d_err, d_best);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

extern "C" int hif8_pts_status(const void* workspace, hif8_stream_t stream)
{
    return hif8_gemm_status(workspace, stream);  // same convention: first int of the workspace
}
