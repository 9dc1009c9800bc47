// Adaptive loss scaling (Section 5.1, "Adaptive Loss-Scaling (ALS)"): the overflow check of the scaled gradients and
// the scale / scale-window controller, both resident on the device so that a training step never waits for the host.
//
// hif8_check_finite streams a tensor once and ORs "has an Inf or NaN" into a device flag; the controller is a
// one-thread kernel over a 64-byte state record.  The scale is a power of two (growth 2, backoff 1/2), so unscaling
// gradients is exponent arithmetic that the conversions and GEMMs of this library already take as device integers.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "hif8.h"
#include "hif8_device.cuh"
#include "hif8_internal.cuh"

namespace hif8 {
extern std::atomic<uint64_t> g_launches;
namespace {

struct AlsState {
    int scale_exp;     // log2 of the loss scale in force
    int window;        // scale window in force (clean iterations before the scale doubles)
    int window_index;  // position in the window list
    int clean;         // clean iterations since the last change of the scale
    int ups;           // increases since the last window change
    int downs;         // decreases not interrupted by an increase
    int steps;         // iterations seen
    int overflows;     // iterations that overflowed
};
static_assert(sizeof(AlsState) <= HIF8_ALS_STATE_BYTES, "state record too large");

__constant__ int c_windows[7] = {1, 20, 50, 100, 200, 500, 1000};

__global__ void als_init_kernel(AlsState* st, int scale_exp, int window_index)
{
    if (threadIdx.x != 0) return;
    st->scale_exp = scale_exp; st->window_index = window_index; st->window = c_windows[window_index];
    st->clean = 0; st->ups = 0; st->downs = 0; st->steps = 0; st->overflows = 0;
}

// one iteration of the controller; consumes and clears the overflow flag
__global__ void als_update_kernel(AlsState* st, int* found_inf)
{
    if (threadIdx.x != 0) return;
    const int overflow = *found_inf != 0;
    *found_inf = 0;
    int se = st->scale_exp, wi = st->window_index, clean = st->clean, ups = st->ups, downs = st->downs;
    if (overflow) {
        if (se > -126) se -= 1;
        clean = 0;
        downs += 1;
        if (downs == 3) { if (wi > 0) wi -= 1; ups = 0; downs = 0; }
    } else {
        clean += 1;
        if (clean >= c_windows[wi]) {
            if (se < 126) se += 1;
            clean = 0;
            ups += 1;
            downs = 0;
            if (ups == 3) { if (wi < 6) wi += 1; ups = 0; downs = 0; }
        }
    }
    st->scale_exp = se; st->window_index = wi; st->window = c_windows[wi]; st->clean = clean; st->ups = ups; st->downs = downs;
    st->steps += 1; st->overflows += overflow;
}

// Exponent field all ones <=> adding one unit of the field's lowest bit to the masked field carries into the bit above
// it: bit 31 for binary32, bits 15 and 31 for two packed 16-bit values (the carry of the low half stops at bit 15).
template <int DT> struct FiniteTraits;
template <> struct FiniteTraits<HIF8_F32>  { static constexpr uint32_t mask = 0x7F800000u, one = 0x00800000u, hit = 0x80000000u; };
template <> struct FiniteTraits<HIF8_BF16> { static constexpr uint32_t mask = 0x7F807F80u, one = 0x00800080u, hit = 0x80008000u; };
template <> struct FiniteTraits<HIF8_F16>  { static constexpr uint32_t mask = 0x7C007C00u, one = 0x04000400u, hit = 0x80008000u; };

template <int DT>
__global__ void __launch_bounds__(kThreads) check_finite_kernel(const void* __restrict__ src, unsigned long long n,
                                                                unsigned long long n_vec, int* found_inf)
{
    using T = FiniteTraits<DT>;
    pdl_launch_dependents();
    pdl_wait_prior_grid();
    uint32_t acc = 0;
    const uint4* v4 = reinterpret_cast<const uint4*>(src);
    for (unsigned long long base = (unsigned long long)blockIdx.x * kThreads * kUnroll; base < n_vec;
         base += (unsigned long long)gridDim.x * kThreads * kUnroll) {
        uint4 v[kUnroll];
#pragma unroll
        for (int j = 0; j < kUnroll; j++) {
            const unsigned long long u = base + (unsigned long long)j * kThreads + threadIdx.x;
            v[j] = u < n_vec ? __ldcs(v4 + u) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < kUnroll; j++)
            acc |= ((v[j].x & T::mask) + T::one) | ((v[j].y & T::mask) + T::one) | ((v[j].z & T::mask) + T::one) |
                   ((v[j].w & T::mask) + T::one);
    }
    // elements not covered by whole vectors (tail, or everything when the pointer is not 16-byte aligned)
    constexpr int PV = DT == HIF8_F32 ? 4 : 8;
    for (unsigned long long i = n_vec * PV + (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < n;
         i += (unsigned long long)gridDim.x * kThreads) {
        const uint32_t w = DT == HIF8_F32 ? reinterpret_cast<const uint32_t*>(src)[i]
                                          : (uint32_t)reinterpret_cast<const unsigned short*>(src)[i];
        acc |= (w & T::mask) + T::one;
    }
    const bool any = __any_sync(0xFFFFFFFFu, (acc & T::hit) != 0);
    if (any && (threadIdx.x & 31) == 0) atomicOr(found_inf, 1);
}

}  // namespace
}  // namespace hif8

using namespace hif8;

extern "C" int hif8_als_state_init(void* d_state, int init_scale_exp, int init_window_index, hif8_stream_t stream)
{
    if (!d_state) return HIF8_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(d_state) & 15u) return HIF8_ERR_ALIGN;
    if (init_scale_exp < -126 || init_scale_exp > 126) return HIF8_ERR_SCALE_RANGE;
    if (init_window_index < 0 || init_window_index > 6) return HIF8_ERR_SHAPE;
    int sms; int rc = checked_device(&sms);
    if (rc) return rc;
    als_init_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(reinterpret_cast<AlsState*>(d_state), init_scale_exp, init_window_index);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

extern "C" int hif8_als_update(void* d_state, int* d_found_inf, hif8_stream_t stream)
{
    if (!d_state || !d_found_inf) return HIF8_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(d_state) & 15u) return HIF8_ERR_ALIGN;
    int sms; int rc = checked_device(&sms);
    if (rc) return rc;
    als_update_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(reinterpret_cast<AlsState*>(d_state), d_found_inf);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}

extern "C" int hif8_check_finite(const void* src, int dtype, size_t n, int* d_found_inf, hif8_stream_t stream)
{
    if (dtype != HIF8_F32 && dtype != HIF8_BF16 && dtype != HIF8_F16) return HIF8_ERR_DTYPE;
    if (!d_found_inf || (n && !src)) return HIF8_ERR_NULL;
    if (n == 0) return HIF8_OK;
    int sms; int rc = checked_device(&sms);
    if (rc) return rc;
    const int pv = dtype == HIF8_F32 ? 4 : 8;
    const size_t item = dtype == HIF8_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(src) & (item - 1)) return HIF8_ERR_ALIGN;
    const unsigned long long n_vec = (reinterpret_cast<uintptr_t>(src) & 15u) ? 0 : n / pv;
    unsigned long long need = n_vec ? (n_vec + (unsigned long long)kThreads * kUnroll - 1) / ((unsigned long long)kThreads * kUnroll)
                                    : (n + kThreads - 1) / kThreads;
    if (!n_vec && need > (unsigned long long)sms * 32) need = (unsigned long long)sms * 32;
    if (need > 0x7FFFFFFFull) need = 0x7FFFFFFFull;
    cudaStream_t st = (cudaStream_t)stream;
    switch (dtype) {
        case HIF8_F32: launch_pdl(check_finite_kernel<HIF8_F32>, (unsigned)need, st, src, (unsigned long long)n, n_vec, d_found_inf); break;
        case HIF8_BF16: launch_pdl(check_finite_kernel<HIF8_BF16>, (unsigned)need, st, src, (unsigned long long)n, n_vec, d_found_inf); break;
        default: launch_pdl(check_finite_kernel<HIF8_F16>, (unsigned)need, st, src, (unsigned long long)n, n_vec, d_found_inf); break;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}
