// GEMM with HiF8 operands decoded in-kernel, for sm_100a (tcgen05 + TMEM + TMA).
//
//   C[m,n] = 2^-(sa+sw) * sum_k value(Aq[m,k]) * value(Wq[k,n])       (Algorithm 1, "MatMul & Restore")
//
// Two paths behind one entry point.  The fused kernel (described next) needs no memory beyond its operands and
// decodes the byte tiles of every CTA in shared memory; because every operand element is then decoded once per
// tile that uses it, it is bound by the decode rate.  With a workspace large enough for both operands in BF16 the
// call decodes each byte once (conversion kernel) and runs the BF16 CTA-pair tensor-core kernel further down.
//
// Every HiF8 value has at most 4 significant bits and an exponent in [-22, 15], so it is exact in BF16 and every
// product of two of them is exact in the FP32 accumulator of the tensor core.
//
// A pair of CTAs (cluster of two, cta_group::2) computes one 256 x 256 tile of C: each CTA stages and decodes its
// own 128 rows of A and 128 columns of W, the even CTA issues the MMAs for both.  Warp roles per CTA:
//   warps 0-3  epilogue: TMEM -> registers -> descale -> BF16 / FP32 -> global
//   warp  4    TMA producer: HiF8 byte tiles (A: 128 x 64, W: 128 x 64 or 64 x 128) into a 4-stage staging ring
//   warp  5    MMA issuer: one elected thread of the even CTA issues tcgen05.mma (256 x 256 x 16 over the pair,
//              BF16 x BF16 -> FP32 in the TMEM of both CTAs)
//   warps 6-21 decode: staging bytes -> BF16; W goes into the canonical 128-byte-swizzled shared-memory operand layout,
//              A ([M,K] form) goes straight into tensor memory (tcgen05.st, one thread per row), from where the MMA
//              reads it as its A operand: the decoded A tile costs neither a shared-memory store nor an operand read
// The operand layout follows the shared-memory matrix descriptor of tcgen05: K-major operands are rows of 64 BF16
// (128 bytes), eight rows form a 1024-byte swizzle atom, 16-byte chunk j of row r is stored at chunk j ^ (r % 8).
// W given as [K, N] is decoded in place as an MN-major operand (atoms of 8 k-rows x 64 n), so no transpose is needed.
//
// Every wait on an mbarrier is bounded; a wait that runs out records a status word, makes all roles leave their
// loops, lets outstanding TMA copies land, frees TMEM and returns.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstring>
#include <mutex>

#include "hif8.h"
#include "hif8_host_cache.h"
#include "hif8_internal.cuh"

namespace hif8 {
extern std::atomic<uint64_t> g_launches;

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kStages8 = 4;    // staging ring of HiF8 byte tiles
constexpr int kStagesBf = 4;   // ring of decoded BF16 operand tiles
constexpr int kStagesBfSwapped = 4, kMaxStagesBf = 8;  // the swapped form (see hif8_gemm_kernel): stages of 128 k, twice the size
constexpr int kEpiWarps = 4, kDecodeWarps = 16;
// The decode warps work in groups, group g on the k-blocks kb = g (mod kDecodeGroups): several k-blocks are in the
// decode stage at once, which covers the latency of each one's lookups, proxy fence and barrier hand-over.  Group g
// owns byte stage g and operand stage g, so every barrier is waited on by one party in program order (a waiter is never
// more than one phase ahead of the barrier, which a parity wait could not tell apart).
constexpr int kDecodeGroups = 4, kGroupWarps = kDecodeWarps / kDecodeGroups, kGroupThreads = kGroupWarps * 32;
static_assert(kStages8 == kDecodeGroups && kStagesBf == kDecodeGroups, "group g owns byte stage g and operand stage g");
// With A decoded into tensor memory the shared memory freed by the A operand tiles can hold either a deeper byte ring
// (8 stages, table with 128-byte rows) or the 64 KiB table whose addresses cost one instruction (4 stages).  Measured at
// 8192 x 28672 x 8192: 4.84 ms against 4.71 ms -- the TMA latency is already covered by four stages, so the wide table is
// the default.
#ifndef HIF8_FUSED_BYTE_STAGES
#define HIF8_FUSED_BYTE_STAGES 4
#endif
#ifndef HIF8_FUSED_WIDE_LUT
#define HIF8_FUSED_WIDE_LUT 1
#endif
constexpr int kStages8Deep = HIF8_FUSED_BYTE_STAGES, kMaxStages8 = 8;  // (barrier slots for up to eight byte stages)
static_assert(kStages8Deep <= kMaxStages8 && kStages8 <= kMaxStages8, "barrier slots");
constexpr bool kWideLut = HIF8_FUSED_WIDE_LUT != 0;
static_assert(kStages8Deep % kDecodeGroups == 0, "a byte stage is always read by the same group");
static_assert(!kWideLut || kStages8Deep == 4, "the 64 KiB table leaves room for four byte stages only");
constexpr int kThreads = (kEpiWarps + 2 + kDecodeWarps) * 32;  // 704
constexpr int kTmaWarp = 4, kMmaWarp = 5, kFirstDecodeWarp = 6;
// per CTA of a pair: 128 rows of A and 128 of the 256 columns of W
constexpr uint32_t kA8Bytes = BM * BK, kB8Bytes = (BN / 2) * BK;            // 8 KiB + 8 KiB
constexpr uint32_t kABfBytes = BM * BK * 2, kBBfBytes = (BN / 2) * BK * 2;  // 16 KiB + 16 KiB
// tensor memory of the fused kernel: columns 0-255 the 128 x 256 FP32 accumulator, then one A operand stage (128 rows x
// 64 BF16 = 32 columns) per operand stage; allocations are powers of two
constexpr uint32_t kTmemColsAcc = 256, kTmemAStageCols = BK / 2, kTmemCols = 512;
static_assert(kTmemColsAcc + kMaxStagesBf * kTmemAStageCols <= kTmemCols, "A operand stages must fit beside the accumulator");
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait

struct SmemLayout {
    static constexpr uint32_t bf = 0;                                                  // 1024-byte aligned atoms
    static constexpr uint32_t u8 = bf + kStagesBf * (kABfBytes + kBBfBytes);           // 96 KiB
    static constexpr uint32_t lut = u8 + kStages8 * (kA8Bytes + kB8Bytes);             // + 64 KiB
    static constexpr uint32_t bars = lut + 256 * 32 * 4;                                // lane-replicated table, 32 KiB
    static constexpr uint32_t n_bars = 2 * kMaxStages8 + 2 * kMaxStagesBf + 1;
    static constexpr uint32_t tmem_slot = bars + n_bars * 8;
    static constexpr uint32_t abort_flag = tmem_slot + 4;
    static constexpr uint32_t total = abort_flag + 4;
};
constexpr uint32_t kSmemBytes = SmemLayout::total + 1024;  // slack for manual 1024-byte alignment
constexpr uint32_t kBarsBytes = 320;                       // barriers, tensor-memory slot, abort flag
static_assert(SmemLayout::n_bars * 8 + 8 <= kBarsBytes, "barrier block");

// ---------------------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false when the barrier did not complete in time or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int where,
                                          unsigned long long limit_ns = kWaitLimitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 1;; it++) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                atomicCAS(status, 0, where);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}

// the same with an L2 eviction policy for the lines the copy brings in
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 32 consecutive columns of this thread's tensor-memory lane (lane field of taddr = first lane of the warp's quarter)
__device__ __forceinline__ void tmem_st_32x32b_x32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- CTA pairs (cluster of two CTAs, cta_group::2)
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Arrival on a barrier of a CTA of the cluster with the default semantics (release at CTA scope).  For the decode warps of
// the fused kernel: what they hand over is read by the tensor core -- tensor memory, ordered by tcgen05.wait::st and
// tcgen05.fence::before_thread_sync, and shared memory, made visible to the async proxy by fence.proxy.async -- not by
// threads of the other CTA.  A release at cluster scope here cost about 2200 cycles per arrival (a per-k-block timeline of
// the groups showed it): it waits for every memory operation the SM has in flight.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA tile load of a CTA pair: data into this CTA's shared memory, completion on a barrier that may live in the peer.
// The tile comes from matrix c2 of a stack of matrices (three-dimensional tensor map, box one matrix deep).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar_cluster)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// one-CTA forms (the narrow kernel)
__device__ __forceinline__ void tc_commit_cta(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// one-CTA form with the A operand (128 rows) in tensor memory
__device__ __forceinline__ void tc_mma_bf16_cta_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)  // arrives on `bar` in both CTAs of the pair
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the same with the A operand in tensor memory (K-major, row i of each CTA's 128 rows in lane i, two BF16 per column)
__device__ __forceinline__ void tc_mma_bf16_pair_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                        uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}


// shared-memory matrix descriptor: start address, leading / stride byte offsets (16-byte units), version 1,
// 128-byte swizzle
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of this architecture
    d |= (uint64_t)2 << 61;  // layout type: 128-byte swizzle
    return d;
}

// BF16 bits of one HiF8 byte (Eq. 1, Eq. 2, specials); used to fill the shared lookup table
__device__ __forceinline__ uint32_t hif8_to_bf16_bits(uint32_t c)
{
    uint32_t sign = (c & 0x80u) << 8, m = c & 0x7Fu;
    if (m == 0) return sign ? 0x7FC0u : 0u;
    if (m == 0x6F) return sign | 0x7F80u;
    if (m < 8) return sign | ((m + 104u) << 7);
    int E; uint32_t M, w;
    if (m < 0x10)      { E = 0; M = m & 7; w = 3; }
    else if (m < 0x20) { E = 1; M = m & 7; w = 3; if (m & 0x08) E = -E; }
    else if (m < 0x40) { E = 2 | ((m >> 3) & 1); M = m & 7; w = 3; if (m & 0x10) E = -E; }
    else if (m < 0x60) { E = 4 | ((m >> 2) & 3); M = m & 3; w = 2; if (m & 0x10) E = -E; }
    else               { E = 8 | ((m >> 1) & 7); M = m & 1; w = 1; if (m & 0x10) E = -E; }
    return sign | ((uint32_t)(E + 127) << 7) | (M << (7 - w));
}

// Fills the decode table: entry (code c, lane l) at word c * ROW_WORDS + l holds the BF16 bits of code c (one copy per
// lane, so that a warp's lookups never meet in a bank).  A warp takes 32 codes: each lane works out one code's value
// once and the warp hands the 32 values round.
template <int ROW_WORDS>
__device__ __forceinline__ void fill_decode_table(uint32_t* table, int warp, int lane, int n_warps)
{
    for (int c0 = warp * 32; c0 < 256; c0 += n_warps * 32) {
        const uint32_t v = hif8_to_bf16_bits((uint32_t)(c0 + lane));
#pragma unroll 8
        for (int k = 0; k < 32; k++) table[(c0 + k) * ROW_WORDS + lane] = __shfl_sync(0xFFFFFFFFu, v, k);
    }
}

// Shared-memory accesses by 32-bit shared-window address: the operand ring lives at a run-time offset inside the dynamic
// allocation, and spelling the state space out keeps every one of these an LDS / STS (never a generic access).
// (not volatile: the table is constant once it is built and every address derives from a byte read after the barrier
// wait, so the compiler is free to issue a whole batch of lookups before the first of them is consumed)
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u16(uint32_t addr, unsigned short v)
{
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// eight HiF8 bytes -> eight BF16 (one 16-byte operand chunk) through the lane-replicated table: lane L only ever touches
// shared-memory bank L, so the lookups of a warp instruction never conflict.  `lut_lane` is the shared address of this
// lane's column.  ROW_SHIFT = 7: rows of 128 bytes, entry of byte c at lut_lane + 128 c (extract, scale, add).
// ROW_SHIFT = 8: rows of 256 bytes in a table that starts on a 64 KiB boundary of the shared window, so that bits 8-15 of
// lut_lane are zero and ONE byte permute drops the code into them: address = lut_lane with byte 1 replaced by c.
template <int ROW_SHIFT>
__device__ __forceinline__ uint4 decode8(uint2 v, uint32_t lut_lane)
{
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const uint32_t w = i < 2 ? v.x : v.y;
        if (ROW_SHIFT == 8) {
            const uint32_t a0 = __byte_perm(w, lut_lane, (i & 1) ? 0x7624 : 0x7604), a1 = __byte_perm(w, lut_lane, (i & 1) ? 0x7634 : 0x7614);
            o[i] = __byte_perm(lds_u32(a0), lds_u32(a1), 0x5410);
        } else {
            const uint32_t c0 = (w >> (16 * (i & 1))) & 0xFFu, c1 = (w >> (16 * (i & 1) + 8)) & 0xFFu;
            o[i] = __byte_perm(lds_u32(lut_lane + c0 * 128), lds_u32(lut_lane + c1 * 128), 0x5410);
        }
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int& tile_m, int& tile_n)
{
    constexpr int kGroupM = 8;  // groups of 8 tile-rows sweep N together: their W tiles stay in L2
    const int per_group = kGroupM * tiles_n;
    const int g = t / per_group, first_m = g * kGroupM;
    const int rows_in_group = min(kGroupM, tiles_m - first_m);
    tile_m = first_m + (t % per_group) % rows_in_group;
    tile_n = (t % per_group) / rows_in_group;
}


// Epilogue of one 32-column chunk of one accumulator row: descale by f1 * f2 (two exact powers of two) and store as
// FP32 or BF16 (round to nearest even); rows / columns outside the matrix are skipped.
__device__ __forceinline__ void store_chunk(const GemmParams& p, int row, int col, const uint32_t (&r)[32], float f1, float f2)
{
    if (row >= p.M || col >= p.N) return;
    const bool full = col + 32 <= p.N;
    if (p.c_is_f32) {
        float* out = reinterpret_cast<float*>(p.C) + (long long)row * p.ldc + col;
        if (full) {
            // C is touched once: streaming loads and stores, so that it does not push operand tiles out of L2; all the
            // loads of the chunk are issued before the first store (they cannot be moved across it by the compiler)
            float4 c[8];
#pragma unroll
            for (int i = 0; i < 8; i++) c[i] = p.accumulate ? __ldcs(reinterpret_cast<const float4*>(out) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int i = 0; i < 8; i++)
                __stcs(reinterpret_cast<float4*>(out) + i,
                       make_float4(__uint_as_float(r[4 * i]) * f1 * f2 + c[i].x, __uint_as_float(r[4 * i + 1]) * f1 * f2 + c[i].y,
                                   __uint_as_float(r[4 * i + 2]) * f1 * f2 + c[i].z, __uint_as_float(r[4 * i + 3]) * f1 * f2 + c[i].w));
        } else {
            // (every index a compile-time constant: a loop that stops at the ragged edge would index the chunk by a
            // variable and put it, for all paths, into local memory -- which has next to no L1 behind it in these kernels)
#pragma unroll
            for (int i = 0; i < 32; i++)
                if (col + i < p.N) out[i] = __uint_as_float(r[i]) * f1 * f2 + (p.accumulate ? out[i] : 0.f);
        }
    } else {
        unsigned short* out = reinterpret_cast<unsigned short*>(p.C) + (long long)row * p.ldc + col;
        uint32_t h[32];
        if (p.accumulate) {  // previous contents of C, widened exactly
            if (full) {
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    const uint4 c = __ldcs(reinterpret_cast<const uint4*>(out + i));
                    h[i] = c.x << 16; h[i + 1] = c.x & 0xFFFF0000u; h[i + 2] = c.y << 16; h[i + 3] = c.y & 0xFFFF0000u;
                    h[i + 4] = c.z << 16; h[i + 5] = c.z & 0xFFFF0000u; h[i + 6] = c.w << 16; h[i + 7] = c.w & 0xFFFF0000u;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; i++) h[i] = (col + i < p.N) ? (uint32_t)out[i] << 16 : 0u;
            }
        }
        uint32_t pk[16];  // two BF16 per word, rounded to nearest even by the conversion instruction (a NaN stays a NaN)
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            float v0 = __uint_as_float(r[i]) * f1 * f2, v1 = __uint_as_float(r[i + 1]) * f1 * f2;
            if (p.accumulate) { v0 += __uint_as_float(h[i]); v1 += __uint_as_float(h[i + 1]); }
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[i >> 1]) : "f"(v1), "f"(v0));  // first source -> upper half
        }
        if (full) {
#pragma unroll
            for (int i = 0; i < 16; i += 4)
                __stcs(reinterpret_cast<uint4*>(out + 2 * i), make_uint4(pk[i], pk[i + 1], pk[i + 2], pk[i + 3]));
        } else {
#pragma unroll
            for (int i = 0; i < 32; i++)
                if (col + i < p.N) out[i] = (unsigned short)(pk[i >> 1] >> (16 * (i & 1)));
        }
    }
}

// The same chunk, descaled and rounded to BF16, into a staging tile in shared memory from which a tile store writes C:
// boxes of 64 columns x 128 rows in the 128-byte-swizzled layout of the tensor map (16-byte piece j of row r sits at
// piece j ^ (r % 8) of its 128-byte line; lines of eight rows form 1024-byte atoms).  `piece0` = first 16-byte piece of
// the chunk within its row of the box (0 or 4).  A thread's four stores hit four different pieces; the eight rows of an
// atom hit eight different ones: no bank conflicts.
__device__ __forceinline__ void stage_chunk_bf16(uint32_t box, int row, int piece0, const uint32_t (&r)[32], float f1, float f2)
{
    const uint32_t line = box + (uint32_t)(row >> 3) * 1024u + (uint32_t)(row & 7) * 128u;
#pragma unroll
    for (int i = 0; i < 4; i++) {
        uint32_t pk[4];
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const float v0 = __uint_as_float(r[8 * i + 2 * j]) * f1 * f2, v1 = __uint_as_float(r[8 * i + 2 * j + 1]) * f1 * f2;
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[j]) : "f"(v1), "f"(v0));
        }
        sts_v4(line + ((uint32_t)((piece0 + i) ^ (row & 7)) << 4), make_uint4(pk[0], pk[1], pk[2], pk[3]));
    }
}
// tile store shared -> global (clipped at the edges of the matrix); the caller commits and waits for the group
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}

// Per-channel weight scales: multiply column col + i of the chunk by 2^-(sa + sw[col + i]).  Lane L fetches the
// exponent of column col + L once; every lane then walks the 32 columns of its own row.
__device__ __forceinline__ void apply_channel_scale(const GemmParams& p, int col, int lane, int sa, uint32_t (&r)[32])
{
    const int mine = (col + lane < p.N) ? -(sa + __ldg(p.d_sw_channel + col + lane)) : 0;
#pragma unroll
    for (int i = 0; i < 32; i++) {
        const int s = __shfl_sync(0xFFFFFFFFu, mine, i);
        const int s1 = s / 2, s2 = s - s1;
        r[i] = __float_as_uint(__uint_as_float(r[i]) * __uint_as_float((uint32_t)(s1 + 127) << 23) *
                               __uint_as_float((uint32_t)(s2 + 127) << 23));
    }
}

// Fused kernel, decode warps: one 128 x 64 tile of HiF8 bytes -> BF16 in the 128-byte-swizzled operand layout, in two
// steps so that the byte tile can be handed back to the TMA producer as soon as it has been read: first a thread's
// eight 8-byte chunks into registers, then lookups and swizzled stores.
constexpr int kChunksPerThread = (BM * BK / 8) / kGroupThreads;  // 8
// K-major source tile [128 rows][64 k]: chunk j (8 codes) of row r -> atom r/8, row r%8, chunk j ^ (r%8).
// MN-major source tile [64 k][128 mn]: chunk (k, mn/8) -> atom (mn/64) * 8 + k/8, row k%8, chunk (mn/8)%8 ^ (k%8).
template <bool MN_MAJOR>
__device__ __forceinline__ void load_tile_chunks(uint32_t src8, int dt, uint2 (&v)[kChunksPerThread])
{
#pragma unroll
    for (int it = 0; it < kChunksPerThread; it++) {
        const int q = it * kGroupThreads + dt;
        v[it] = MN_MAJOR ? lds_v2(src8 + (q >> 4) * BM + (q & 15) * 8) : lds_v2(src8 + (q >> 3) * BK + (q & 7) * 8);
    }
}
template <bool MN_MAJOR, int ROW_SHIFT = 7>
__device__ __forceinline__ void decode_tile_chunks(const uint2 (&v)[kChunksPerThread], uint32_t dst, int dt, uint32_t lut)
{
#pragma unroll
    for (int it = 0; it < kChunksPerThread; it++) {
        const int q = it * kGroupThreads + dt;
        if (MN_MAJOR) {
            const int k = q >> 4, jn = q & 15, atom = (jn >> 3) * 8 + (k >> 3);
            sts_v4(dst + atom * 1024 + (k & 7) * 128 + (((jn & 7) ^ (k & 7)) << 4), decode8<ROW_SHIFT>(v[it], lut));
        } else {
            const int r = q >> 3, j = q & 7;
            sts_v4(dst + (r >> 3) * 1024 + (r & 7) * 128 + ((j ^ (r & 7)) << 4), decode8<ROW_SHIFT>(v[it], lut));
        }
    }
}

// Shared memory of the fused kernel.
// A given as [K,M] (decoded into shared memory): the fixed layout of SmemLayout.
// A given as [M,K] (decoded into tensor memory): no A operand tiles, and the lookup table has rows of 256 bytes and starts on
// a 64 KiB boundary of the shared window (see decode8).  Everything else is dealt out in 16 KiB slots around the table: as
// many as fit in front of it, the rest behind it.  Slots 0-3: W operand stages, slots 4-7: byte stages (A 8 KiB + W 8 KiB).
constexpr uint32_t kSlotBytes = 16384, kLutBytesWide = 65536, kLutBytesNarrow = 256 * 32 * 4, kFusedSlots = kStagesBf + kStages8Deep;
static_assert(kBBfBytes == kSlotBytes && kA8Bytes + kB8Bytes == kSlotBytes, "one stage per slot");
constexpr uint32_t kSmemBytesWide = 227 * 1024;  // the whole opt-in maximum; the kernel checks that its plan fits

// PLAN 0: slots around the 64 KiB table.  1: the layout of SmemLayout (A operand tiles in shared memory).  2: the swapped
// form -- eight operand stages of 16 KiB, four byte stages of 8 KiB, the 32 KiB table, barriers, one after the other.
constexpr int kStages8Swapped = 4;  // byte stages of the swapped form (A bytes only, 128 k: 16 KiB each)
constexpr uint32_t kSmemBytesSwapped = kStagesBfSwapped * 2 * kBBfBytes + kStages8Swapped * 2 * kA8Bytes + 256 * 32 * 4 + kBarsBytes + 1024;
template <int PLAN>
struct FusedSmem {
    static constexpr bool FIXED = PLAN == 1;
    uint32_t base, lut, bars, behind;  // shared-window addresses; base is 1024-byte aligned
    int n_front;                       // slots in front of the table
    uint32_t end;                      // first byte behind everything

    __device__ explicit FusedSmem(uint32_t raw)
    {
        base = (raw + 1023u) & ~1023u;
        if (FIXED) {
            lut = base + SmemLayout::lut; bars = base + SmemLayout::bars; behind = 0; n_front = 0; end = base + SmemLayout::total;
        } else if (PLAN == 2) {
            behind = 0; n_front = 2 * kStagesBfSwapped;
            lut = base + kStagesBfSwapped * 2 * kBBfBytes + kStages8Swapped * 2 * kA8Bytes; bars = lut + kLutBytesNarrow; end = bars + kBarsBytes;
        } else if (!kWideLut) {
            // table with rows of 128 bytes: no alignment to honour, everything in a row: slots, table, barriers
            n_front = (int)kFusedSlots; behind = 0;
            lut = base + kFusedSlots * kSlotBytes; bars = lut + kLutBytesNarrow; end = bars + kBarsBytes;
        } else {
            lut = (base + kLutBytesWide - 1) & ~(kLutBytesWide - 1);
            const uint32_t front = lut - base;
            n_front = (int)min(front / kSlotBytes, kFusedSlots);
            behind = lut + kLutBytesWide;
            const uint32_t after_slots = behind + (kFusedSlots - n_front) * kSlotBytes;
            // barriers, tensor-memory slot and abort flag (256 bytes): in the gap in front of the table if there is one
            bars = (front - n_front * kSlotBytes >= kBarsBytes) ? base + n_front * kSlotBytes : after_slots;
            end = bars >= after_slots ? bars + kBarsBytes : after_slots;
        }
    }
    __device__ uint32_t slot(int i) const { return i < n_front ? base + (uint32_t)i * kSlotBytes : behind + (uint32_t)(i - n_front) * kSlotBytes; }
    __device__ uint32_t a_bf(int s) const { return base + SmemLayout::bf + s * (kABfBytes + kBBfBytes); }                       // FIXED only
    __device__ uint32_t w_bf(int s) const { return PLAN == 2 ? base + (uint32_t)s * 2 * kBBfBytes : (FIXED ? a_bf(s) + kABfBytes : slot(s)); }
    __device__ uint32_t a_u8(int s) const
    {
        if (PLAN == 2) return base + kStagesBfSwapped * 2 * kBBfBytes + (uint32_t)s * 2 * kA8Bytes;
        return FIXED ? base + SmemLayout::u8 + s * (kA8Bytes + kB8Bytes) : slot(kStagesBf + s);
    }
    // staging box j (16 KiB) of the result tile: the operand stages, idle once the accumulator is complete
    __device__ uint32_t box(int j) const { return FIXED ? base + SmemLayout::bf + (uint32_t)j * kSlotBytes : slot(j); }
    __device__ uint32_t w_u8(int s) const { return a_u8(s) + kA8Bytes; }
    __device__ uint32_t tmem_slot() const { return bars + SmemLayout::n_bars * 8; }
    __device__ uint32_t abort_flag() const { return tmem_slot() + 4; }
};

// A_MODE 0: A given as [M,K] bytes, decoded into tensor memory.  1: A given as [K,M] bytes, decoded into shared memory
// (MN-major operand).  2: A already expanded to BF16 [M,K] in the caller's workspace (only W is decoded here): its tiles
// come by TMA straight into the K-major operand stages, completing on the leader's "operands ready" barrier.
// SWAPPED (with A_MODE 0 and W_IS_NK): the kernel computes C^T = W^T A^T.  Its byte operand -- rows decoded into tensor
// memory -- is the caller's [N,K] weight, its shared-memory operand the caller's activations, already expanded to BF16
// [M,K] and brought by TMA; nothing decoded here is stored to shared memory or read back from it by the tensor core.  The
// kernel's "M" is the caller's N and vice versa, and the epilogue writes the accumulator transposed.
template <int A_MODE, bool W_IS_NK, bool SWAPPED = false>
__global__ void __launch_bounds__(kThreads, 1)
hif8_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                 const __grid_constant__ CUtensorMap map_c, const GemmParams p)
{
    extern __shared__ unsigned char smem_raw[];
    constexpr bool A_IS_KM = A_MODE == 1, A_BF16 = A_MODE == 2, kFixed = A_MODE != 0;
    static_assert(!SWAPPED || (A_MODE == 0 && W_IS_NK), "the swapped form reads both operands K-major");
    constexpr int kLutShift = (kFixed || SWAPPED || !kWideLut) ? 7 : 8;
    constexpr int kS8 = SWAPPED ? kStages8Swapped : (kFixed ? kStages8 : kStages8Deep);  // depth of the byte ring
    // operand stages: one per decode group, or (SWAPPED: nothing decoded goes to shared memory, which leaves the room) two, so
    // that a group starts its next k-block while the MMAs of its last one are still queued behind the other groups'
    constexpr int kSB = SWAPPED ? kStagesBfSwapped : kStagesBf;
    const FusedSmem<SWAPPED ? 2 : (kFixed ? 1 : 0)> plan(smem_u32(smem_raw));
    const uint32_t base = plan.base;
    unsigned char* sm = smem_raw - smem_u32(smem_raw);  // generic pointer of shared-window address 0
    {
        uint32_t dyn_bytes;
        asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_bytes));
        if (plan.end > smem_u32(smem_raw) + dyn_bytes) {  // the plan does not fit (the same answer in every thread of the pair)
            if (threadIdx.x == 0) atomicCAS(p.status, 0, 7);
            return;
        }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0: leader of the pair (issues the MMAs), 1: peer
    const bool leader = rank == 0;

    const uint32_t bars = plan.bars;
    auto bar_u8_full = [&](int s) { return bars + 8u * s; };                                   // per CTA
    auto bar_u8_empty = [&](int s) { return bars + 8u * (kMaxStages8 + s); };                     // per CTA
    auto bar_bf_full = [&](int s) { return bars + 8u * (2 * kMaxStages8 + s); };                  // leader: both CTAs' decode warps
    auto bar_bf_empty = [&](int s) { return bars + 8u * (2 * kMaxStages8 + kMaxStagesBf + s); };  // per CTA, leader's commits
    const uint32_t bar_acc_full = bars + 8u * (2 * kMaxStages8 + 2 * kMaxStagesBf);                  // per CTA, leader's commit
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + plan.abort_flag());
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + plan.tmem_slot());
    uint32_t* lut_all = reinterpret_cast<uint32_t*>(sm + plan.lut);
    const uint32_t lut = plan.lut + 4u * lane;  // this lane's column of the table

    // 256 x 256 tile of this pair (groups of 8 tile-rows share their W tiles in L2); this CTA: 128 rows, 128 columns of W
    int tile_m, tile_n;
    tile_coords((int)(blockIdx.x >> 1), (p.M + 2 * BM - 1) / (2 * BM), p.tiles_n, tile_m, tile_n);
    const int m0 = tile_m * 2 * BM + (int)rank * BM, n0 = tile_n * BN, nh = n0 + (int)rank * (BN / 2);
    // k per operand stage: 64, or (SWAPPED) 128 -- one hand-over, one commit and one probe by the MMA thread per 128 k
    constexpr int KB = SWAPPED ? 2 * BK : BK;
    const int num_kb = (p.K + KB - 1) / KB;

    // ---- set-up
    fill_decode_table<(1 << (kLutShift - 2))>(lut_all, warp, lane, kThreads / 32);  // rows of 1 << kLutShift bytes
    if (threadIdx.x == 0) {
        for (int s = 0; s < kS8; s++) { mbar_init(bar_u8_full(s), 1); mbar_init(bar_u8_empty(s), kGroupWarps); }
        // operands ready: both CTAs' decode group, plus (A_BF16) the leader's announcement of the A tile bytes
        for (int s = 0; s < kSB; s++) { mbar_init(bar_bf_full(s), 2 * kGroupWarps + ((A_BF16 || SWAPPED) ? 1 : 0)); mbar_init(bar_bf_empty(s), 1); }
        mbar_init(bar_acc_full, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {  // this warp owns the TMEM allocation (both CTAs of the pair take part)
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(plan.tmem_slot()), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // barriers of both CTAs exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if ((A_BF16 || SWAPPED) && warp == 0) {
        // ------------------------------------------------------------------ second producer (an epilogue warp, idle until the
        // accumulator is complete): the BF16 tiles of the operand that was expanded beforehand.  Issuing a tile copy costs its
        // thread a few hundred cycles, and with both kinds of copy on one thread that thread set the pace.  The tile of k-block
        // kb goes straight into operand stage sb (this CTA's 128 rows) once the MMAs of its previous use have read it; both
        // CTAs' copies complete on the leader's "operands ready" barrier, which the leader arms with the bytes of both.
        if (lane == 0) {
            for (int kb = 0; kb < num_kb; kb++) {
                const int sb = kb % kSB, rb = kb / kSB;
                if (rb > 0 && !mbar_wait(bar_bf_empty(sb), (rb - 1) & 1, abort_flag, p.status, 6)) break;
                if (*abort_flag) break;
                if (leader) mbar_arrive_expect_tx(bar_bf_full(sb), SWAPPED ? 4 * kBBfBytes : 2 * kABfBytes);
                if (SWAPPED) {  // 128 k of BF16 are two boxes of 64 (the swizzle span), into the two halves of the stage
                    tma_load_3d_pair(plan.w_bf(sb), &map_w, kb * KB, nh, 0, map_to_cta(bar_bf_full(sb), 0));
                    tma_load_3d_pair(plan.w_bf(sb) + kBBfBytes, &map_w, kb * KB + BK, nh, 0, map_to_cta(bar_bf_full(sb), 0));
                } else tma_load_3d_pair(plan.a_bf(sb), &map_a, kb * BK, m0, 0, map_to_cta(bar_bf_full(sb), 0));
            }
        }
        __syncwarp();
    }
    if (warp == kTmaWarp) {
        // ------------------------------------------------------------------ TMA producer (each CTA feeds itself)
        if (lane == 0) {
            int issued = 0;
            for (int kb = 0; kb < num_kb; kb++) {
                const int s = kb % kS8, round = kb / kS8;
                if (round > 0 && !mbar_wait(bar_u8_empty(s), (round - 1) & 1, abort_flag, p.status, 1)) break;
                if (*abort_flag) break;
                const uint32_t dst_a = plan.a_u8(s), dst_b = plan.w_u8(s);
                mbar_arrive_expect_tx(bar_u8_full(s), (A_BF16 ? 0u : (SWAPPED ? 2 * kA8Bytes : kA8Bytes)) + (SWAPPED ? 0u : kB8Bytes));
                if (A_IS_KM) tma_load_2d(dst_a, &map_a, m0, kb * BK, bar_u8_full(s));
                else if (!A_BF16) tma_load_2d(dst_a, &map_a, kb * KB, m0, bar_u8_full(s));  // (SWAPPED: one box of 128 k)
                if (SWAPPED) {}
                else if (W_IS_NK) tma_load_2d(dst_b, &map_w, kb * BK, nh, bar_u8_full(s));
                else tma_load_2d(dst_b, &map_w, nh, kb * BK, bar_u8_full(s));
                issued = kb + 1;
            }
            if (*abort_flag) {
                // let the copies already issued land before this CTA's shared memory goes away
                for (int kb = max(0, issued - kS8); kb < issued; kb++) {
                    const int s = kb % kS8;
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_u8_full(s), (kb / kS8) & 1) && global_ns() - t0 < kWaitLimitNs) {}
                }
                if (A_BF16 || SWAPPED) {  // (the BF16 tiles complete on a barrier that also counts the decode groups, which have given up:
                               // their copies get a fixed 50 us instead)
                    const unsigned long long t0 = global_ns();
                    while (global_ns() - t0 < 50000ull) {}
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            // instruction descriptor: FP32 accumulator, BF16 A and B, A K-major, B K- or MN-major, N = 256, M = 256 (pair)
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_IS_KM ? 1u : 0u) << 15) | ((W_IS_NK ? 0u : 1u) << 16) |
                                   ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
            // An MMA is accepted only when the tensor pipe has room, so whatever this thread does between two of them leaves
            // the pipe idle: the barrier of the next k-block is probed, and its addresses are formed, between the third and
            // the fourth MMA of the current one (while the third runs), not after the commit.
            bool ok = mbar_wait(bar_bf_full(0), 0, abort_flag, p.status, 2);
            uint32_t a_addr = plan.a_bf(0), b_addr = plan.w_bf(0), a_tmem = tmem_base + kTmemColsAcc;
            for (int kb = 0; kb < num_kb && ok; kb++) {
                const int s = kb % kSB;
                tc_fence_after();
                bool next_ready = true;
                uint32_t a_next = 0, b_next = 0, t_next = 0;
#pragma unroll
                for (int kk = 0; kk < KB / 16; kk++) {
                    if (kk == KB / 16 - 1 && kb + 1 < num_kb) {
                        const int sn = (kb + 1) % kSB;
                        next_ready = mbar_try_wait(bar_bf_full(sn), (uint32_t)(((kb + 1) / kSB) & 1));
                        a_next = plan.a_bf(sn); b_next = plan.w_bf(sn);
                        t_next = tmem_base + kTmemColsAcc + (uint32_t)(sn * (KB / 2));
                    }
                    // K-major: 16 k = 32 bytes inside the 128-byte row (SWAPPED: the second 64 k are the stage's second half);
                    // MN-major: 16 k = two 1024-byte atoms
                    const uint64_t db = W_IS_NK ? make_smem_desc(b_addr + (kk >> 2) * kBBfBytes + (kk & 3) * 32, 16, 1024)
                                                : make_smem_desc(b_addr + kk * 2048, 8192, 1024);
                    if (A_IS_KM) {
                        tc_mma_bf16_pair(tmem_base, make_smem_desc(a_addr + kk * 2048, 8192, 1024), db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                    } else if (A_BF16) {
                        tc_mma_bf16_pair(tmem_base, make_smem_desc(a_addr + kk * 32, 16, 1024), db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                    } else {
                        // A from tensor memory: stage s, 16 k = 8 columns
                        tc_mma_bf16_pair_a_tmem(tmem_base, a_tmem + (uint32_t)(kk * 8), db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                    }
                }
                tc_commit_pair(bar_bf_empty(s));  // frees this operand stage in both CTAs once the MMAs have read it
                if (kb + 1 < num_kb) {
                    if (!next_ready) ok = mbar_wait(bar_bf_full((kb + 1) % kSB), (uint32_t)(((kb + 1) / kSB) & 1), abort_flag, p.status, 2);
                    a_addr = a_next; b_addr = b_next; a_tmem = t_next;
                }
            }
            if (ok) tc_commit_pair(bar_acc_full);
        }
    } else if (warp >= kFirstDecodeWarp) {
        // ------------------------------------------------------------------ decode warps
        const int group = (warp - kFirstDecodeWarp) / kGroupWarps;
        const int dt = threadIdx.x - (kFirstDecodeWarp + group * kGroupWarps) * 32;  // 0..kGroupThreads-1
        bool ok = true;
        for (int kb = group; kb < num_kb && ok; kb += kDecodeGroups) {
            const int s8 = kb % kS8, r8 = kb / kS8, sb = kb % kSB, rb = kb / kSB;
            ok = mbar_wait(bar_u8_full(s8), r8 & 1, abort_flag, p.status, 3);
            if (ok && rb > 0) ok = mbar_wait(bar_bf_empty(sb), (rb - 1) & 1, abort_flag, p.status, 4);
            if (!ok) break;
            const uint32_t a8 = plan.a_u8(s8), b8 = plan.w_u8(s8);
            const uint32_t abf = plan.a_bf(sb), bbf = plan.w_bf(sb);
            uint2 vw[kChunksPerThread];
            if (A_IS_KM) {
                uint2 va[kChunksPerThread];
                load_tile_chunks<true>(a8, dt, va);
                load_tile_chunks<!W_IS_NK>(b8, dt, vw);
                __syncwarp();  // every lane's reads of the byte stage are done: the producer may refill it during the decode
                if (lane == 0) mbar_arrive(bar_u8_empty(s8));
                decode_tile_chunks<true, kLutShift>(va, abf, dt, lut);
            } else if (A_BF16) {
                // A was expanded beforehand and arrives by TMA: only the W tile is decoded here
                load_tile_chunks<!W_IS_NK>(b8, dt, vw);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_u8_empty(s8));
            } else if (SWAPPED) {
                // As below, with rows of 128 k: the byte tile arrives with the 128-byte TMA swizzle (chunk j of row r at chunk
                // j ^ (r & 7)), the row is decoded in two halves of 64 into the two halves of the 64-column stage.
                const int quarter = warp & 3, r = quarter * 32 + lane;
                const uint32_t a_row = a8 + (uint32_t)r * KB, sw = (uint32_t)r & 7u;
                uint4 va[KB / 16];
#pragma unroll
                for (int j = 0; j < KB / 16; j++) va[j] = lds_v4(a_row + (((uint32_t)j ^ sw) << 4));
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_u8_empty(s8));
#pragma unroll
                for (int half = 0; half < 2; half++) {
                    uint32_t o[BK / 2];
#pragma unroll
                    for (int j = 0; j < BK / 16; j++) {
                        const uint4 v = va[half * (BK / 16) + j];
                        const uint4 lo = decode8<kLutShift>(make_uint2(v.x, v.y), lut), hi = decode8<kLutShift>(make_uint2(v.z, v.w), lut);
                        o[8 * j + 0] = lo.x; o[8 * j + 1] = lo.y; o[8 * j + 2] = lo.z; o[8 * j + 3] = lo.w;
                        o[8 * j + 4] = hi.x; o[8 * j + 5] = hi.y; o[8 * j + 6] = hi.z; o[8 * j + 7] = hi.w;
                    }
                    tmem_st_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + kTmemColsAcc + (uint32_t)(sb * (KB / 2) + half * (BK / 2)), o);
                }
            } else {
                // A [M,K]: this thread owns row (its warp's quarter of the 128 tensor-memory lanes) * 32 + lane.  The byte
                // tile arrives with the 64-byte TMA swizzle (16-byte chunk j of row r sits at chunk j ^ ((r >> 1) & 3)), so
                // the lanes of a warp, 64 bytes apart, read their chunk j from different banks.
                const int quarter = warp & 3, r = quarter * 32 + lane;
                const uint32_t a_row = a8 + (uint32_t)r * BK, sw = (uint32_t)(r >> 1) & 3u;
                uint4 va[BK / 16];
#pragma unroll
                for (int j = 0; j < BK / 16; j++) va[j] = lds_v4(a_row + (((uint32_t)j ^ sw) << 4));
                load_tile_chunks<!W_IS_NK>(b8, dt, vw);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_u8_empty(s8));
                uint32_t o[BK / 2];  // 64 BF16 of this row, two per column
#pragma unroll
                for (int j = 0; j < BK / 16; j++) {
                    const uint4 lo = decode8<kLutShift>(make_uint2(va[j].x, va[j].y), lut), hi = decode8<kLutShift>(make_uint2(va[j].z, va[j].w), lut);
                    o[8 * j + 0] = lo.x; o[8 * j + 1] = lo.y; o[8 * j + 2] = lo.z; o[8 * j + 3] = lo.w;
                    o[8 * j + 4] = hi.x; o[8 * j + 5] = hi.y; o[8 * j + 6] = hi.z; o[8 * j + 7] = hi.w;
                }
                tmem_st_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + kTmemColsAcc + (uint32_t)(sb * kTmemAStageCols), o);
            }
            if (!SWAPPED) decode_tile_chunks<!W_IS_NK, kLutShift>(vw, bbf, dt, lut);
            if (A_MODE == 0) tmem_st_wait();  // the row is in tensor memory
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // make the stores visible to the tensor core
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(map_to_cta(bar_bf_full(sb), 0));  // the leader's MMAs read both CTAs' operands
        }
    }
    if (warp != kTmaWarp && warp != kMmaWarp) {
        // ------------------------------------------------------------------ epilogue (each CTA drains its rows)
        // Warps 0-3 and, once their k-blocks are done, the sixteen decode warps: a warp reaches the quarter (warp % 4) of
        // the tensor-memory lanes, so every quarter has five warps, which share its eight 32-column chunks (the drain is
        // not overlapped with anything: with four warps it took a tenth of the tile's time).
        const int quarter = warp & 3;
        const int share = warp < kEpiWarps ? 0 : (warp - quarter) / 4 - (quarter < 2 ? 1 : 0);  // 0..4 within the quarter
        static_assert(kEpiWarps == 4 && kTmaWarp == 4 && kMmaWarp == 5 && kFirstDecodeWarp == 6 && kDecodeWarps == 16,
                      "five warps per lane quarter: w, and w + 4k without the two single-thread warps");
        const bool ok = mbar_wait(bar_acc_full, 0, abort_flag, p.status, 5);
        if (ok) {
            tc_fence_after();
            const int sa = p.d_sa ? *p.d_sa : 0;
            const int s = p.d_sw_channel ? 0 : -(sa + (p.d_sw ? *p.d_sw : 0));
            const int s1 = s / 2, s2 = s - s1;  // |s1|, |s2| <= 126: two exact power-of-two factors
            const float f1 = __uint_as_float((uint32_t)(s1 + 127) << 23), f2 = __uint_as_float((uint32_t)(s2 + 127) << 23);
            const int row = m0 + quarter * 32 + lane;
            // (separate loops rather than branches inside one: the register allocation of each stays that of its own path)
            if (SWAPPED) {
                // accumulator row = the caller's column n (one weight exponent per thread), accumulator column = the caller's
                // row m: for every m the warp writes 32 consecutive n
                const int sw = p.d_sw_channel ? (row < p.M ? __ldg(p.d_sw_channel + row) : 0) : (p.d_sw ? *p.d_sw : 0);
                const int sc = -(sa + sw), t1 = sc / 2, t2 = sc - t1;
                const float g1 = __uint_as_float((uint32_t)(t1 + 127) << 23), g2 = __uint_as_float((uint32_t)(t2 + 127) << 23);
                if (p.c_by_tma) {
                    // BF16 result that replaces C: into the staging boxes of the tile stores (64 of the caller's columns x 128
                    // of its rows each, 128-byte-swizzled; box = column half + 2 * row half of this CTA's 256 x 128 piece).  For
                    // one row m the 32 lanes write 32 consecutive columns: 64 contiguous bytes of one line.
                    const int nl = quarter * 32 + lane;
                    const uint32_t piece = (uint32_t)((nl & 63) >> 3), within = (uint32_t)(nl & 7) * 2u;
#pragma unroll 1
                    for (int c = share * 32; c < BN; c += 5 * 32) {
                        uint32_t r[32];
                        tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + c, r);
                        tmem_ld_wait();
                        const uint32_t box = plan.box((nl >> 6) + 2 * (c >> 7));
#pragma unroll
                        for (int i = 0; i < 32; i++) {
                            const uint32_t rr = (uint32_t)((c + i) & 127);
                            unsigned short b;
                            asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(b) : "f"(__uint_as_float(r[i]) * g1 * g2));
                            sts_u16(box + (rr >> 3) * 1024u + (rr & 7u) * 128u + ((piece ^ (rr & 7u)) << 4) + within, b);
                        }
                    }
                } else
#pragma unroll 1
                for (int c = share * 32; c < BN; c += 5 * 32) {
                    uint32_t r[32];
                    tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + c, r);
                    tmem_ld_wait();
                    if (row < p.M) {
#pragma unroll
                        for (int i = 0; i < 32; i++) {
                            const int m = n0 + c + i;
                            if (m < p.N) {
                                float v = __uint_as_float(r[i]) * g1 * g2;
                                if (p.c_is_f32) {
                                    float* out = reinterpret_cast<float*>(p.C) + (long long)m * p.ldc + row;
                                    *out = p.accumulate ? v + *out : v;
                                } else {
                                    unsigned short* out = reinterpret_cast<unsigned short*>(p.C) + (long long)m * p.ldc + row;
                                    if (p.accumulate) v += __uint_as_float((uint32_t)*out << 16);
                                    unsigned short b;
                                    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(b) : "f"(v));
                                    *out = b;
                                }
                            }
                        }
                    }
                }
            } else if (!A_IS_KM && p.c_by_tma) {
#pragma unroll 1
                for (int c = share * 32; c < BN; c += 5 * 32) {
                    uint32_t r[32];
                    tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + c, r);
                    tmem_ld_wait();
                    if (p.d_sw_channel) apply_channel_scale(p, n0 + c, lane, sa, r);
                    // the operand stages are idle once the accumulator is complete: box c / 64 of the result tile goes there
                    stage_chunk_bf16(plan.box(c >> 6), quarter * 32 + lane, (c & 63) >> 3, r, f1, f2);
                }
            } else {
#pragma unroll 1
                for (int c = share * 32; c < BN; c += 5 * 32) {
                    uint32_t r[32];
                    tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + c, r);
                    tmem_ld_wait();
                    if (p.d_sw_channel) apply_channel_scale(p, n0 + c, lane, sa, r);
                    store_chunk(p, row, n0 + c, r, f1, f2);
                }
            }
        }
        if (!A_IS_KM && p.c_by_tma) {
            // Stores of 16 bytes per lane to 32 different rows made the drain as slow as one L2 transaction per clock allows
            // (4096 of them per CTA); four tile stores write whole lines instead.  All twenty warps meet (named barrier 1),
            // then one thread issues the stores and waits until shared memory has been read.
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            asm volatile("bar.sync 1, %0;" ::"n"((kEpiWarps + kDecodeWarps) * 32) : "memory");
            if (threadIdx.x == 0 && ok && !*abort_flag) {
                if (SWAPPED) {  // x = the caller's column (this CTA's 128, two boxes), y = its row (256, two boxes)
#pragma unroll
                    for (int j = 0; j < 4; j++) tma_store_2d(&map_c, plan.box(j), m0 + (j & 1) * 64, n0 + (j >> 1) * 128);
                } else {
#pragma unroll
                    for (int j = 0; j < BN / 64; j++) tma_store_2d(&map_c, plan.box(j), n0 + j * 64, m0);
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            }
        }
    }

    // ---- teardown: all waits are bounded, so everybody arrives; nobody leaves while the peer may still read this
    // CTA's operands or signal its barriers; then the allocating warps free TMEM
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------------------
// Narrow products (M <= 64 rows of activations: the decode phase of inference).  The product is bound by reading the
// weight bytes once, so the roles are swapped: a CTA streams a slab of 128 weight columns as the 128-row MMA operand and
// the few activation rows are the narrow operand (MMA N = M rounded up to 16).  One CTA per SM, no pairs:
//   warp 4        copies: per pair block (two k-blocks) one tile of weight bytes and one of activation bytes
//                 (activations expanded to BF16 beforehand, when the workspace has room: their tiles instead, one per
//                 k-block, straight into the operand stages; the groups then decode weights only)
//   warps 6-21    four decode groups, group g on the k-blocks it = g (mod 4): a thread owns one weight column of the slab,
//                 decodes its 64 bytes of the k-block and stores them as its lane of a weight stage in tensor memory (the A
//                 operand of tcgen05.mma may live there); the group also decodes the activation tile into shared memory
//   warps 5, 22-24  MMA issuers (below)
//   warps 0-3     epilogue
// The accumulator holds C transposed (row = weight column n, column = activation row m); the epilogue writes C[m][n] with
// consecutive lanes on consecutive n.
// ---------------------------------------------------------------------------------------------------------
constexpr int kNarrowMaxM = 64;
constexpr uint32_t kNwW8 = BM * BK, kNwA8 = kNarrowMaxM * BK;          // byte tiles per stage: 8 KiB weights, 4 KiB activations
constexpr uint32_t kNwABf = kNarrowMaxM * BK * 2;  // activation operand tile per stage: 8 KiB (the weights go to tensor memory)
// A copy brings two k-blocks (a "pair block": 128 bytes of k) of weights and of activations: issuing a tile copy costs
// its thread a few hundred cycles whatever the size, and with one copy of each kind per k-block that thread set the pace.
// Four stages of 16 KiB + 8 KiB: 64 KiB of weights in flight per SM (a fifth stage changed nothing).
constexpr int kNwByteStages = 4, BK2 = 2 * BK;
// Operand stages (32 tensor-memory columns of weights + 8 KiB of activations in shared memory each): two per group, so
// that a group starts its next k-block without waiting for the MMAs of its previous one
constexpr int kNwTmemStages = 2 * kDecodeGroups;
struct SmemLayoutN {
    static constexpr uint32_t bf = 0;
    static constexpr uint32_t u8 = bf + kNwTmemStages * kNwABf;
    static constexpr uint32_t lut = u8 + kNwByteStages * 2 * (kNwW8 + kNwA8);
    static constexpr uint32_t bars = lut + 256 * 32 * 4;
    static constexpr uint32_t n_bars = 2 * kNwByteStages + 2 * kNwTmemStages + 4;
    static constexpr uint32_t tmem_slot = bars + n_bars * 8;
    static constexpr uint32_t abort_flag = tmem_slot + 4;
    static constexpr uint32_t total = abort_flag + 4;
};
constexpr uint32_t kSmemBytesN = SmemLayoutN::total + 1024;
// Where the narrow kernel keeps what.  WIDE = false: the fixed layout above.  WIDE = true ([N,K] weights with the activations
// expanded beforehand: the byte stages hold weights only, 16 KiB each): the decode table has rows of 256 bytes and starts on a 64 KiB boundary
// of the shared window, so that one byte permute makes a lookup's address (see decode8); as many operand stages (8 KiB) as
// fit lie in front of it, the other operand stages, the byte stages and the barriers behind it.
template <bool WIDE>
struct NarrowSmem {
    uint32_t base, lut, bars, end;  // shared-window addresses; base is 1024-byte aligned
    uint32_t behind, u8_0;
    int n_front;
    __device__ explicit NarrowSmem(uint32_t raw)
    {
        base = (raw + 1023u) & ~1023u;
        if (!WIDE) {
            lut = base + SmemLayoutN::lut; bars = base + SmemLayoutN::bars; end = base + SmemLayoutN::total;
            behind = 0; u8_0 = base + SmemLayoutN::u8; n_front = kNwTmemStages;
        } else {
            lut = (base + kLutBytesWide - 1) & ~(kLutBytesWide - 1);
            n_front = (int)min((lut - base) / kNwABf, (uint32_t)kNwTmemStages);
            behind = lut + kLutBytesWide;
            u8_0 = behind + (uint32_t)(kNwTmemStages - n_front) * kNwABf;
            bars = u8_0 + kNwByteStages * 2 * kNwW8;
            end = bars + SmemLayoutN::n_bars * 8 + 8;
        }
    }
    __device__ uint32_t bf(int s) const { return s < n_front ? base + (uint32_t)s * kNwABf : behind + (uint32_t)(s - n_front) * kNwABf; }
    __device__ uint32_t u8(int s) const { return u8_0 + (uint32_t)s * (WIDE ? 2 * kNwW8 : 2 * (kNwW8 + kNwA8)); }
    __device__ uint32_t tmem_slot() const { return bars + SmemLayoutN::n_bars * 8; }
    __device__ uint32_t abort_flag() const { return tmem_slot() + 4; }
};
// Tensor memory: the accumulators (two per issuer: the epilogue of one segment overlaps the next segment's MMAs), then
// one weight stage (128 rows x 64 BF16 = 32 columns) per operand stage.
// MMA issuers.  One thread that waits for a stage, issues its four MMAs and commits spends about a thousand cycles per
// k-block, more than the decode groups or the copies need; so up to four threads (one per warp) share the k-blocks,
// issuer q taking the k-blocks it = q (mod issuers) into accumulators of its own, which the epilogue adds.  Up to 32
// activation rows every issuer has two accumulators; above that either four issuers with one accumulator each or two with
// two (the kernel says which): issuers x buffers x rows stays within 256 columns.
constexpr int kNwMaxIssuers = 4;
constexpr int kThreadsN = kThreads + (kNwMaxIssuers - 1) * 32;  // 800: the first issuer is the MMA warp of the other kernels
constexpr uint32_t kTmemAccN = 2 * 2 * kNarrowMaxM, kTmemColsN = 512;
static_assert(kTmemAccN + kNwTmemStages * (BK / 2) <= kTmemColsN, "weight stages fit beside the accumulators");
static_assert(2 * kNwMaxIssuers * 32 <= kTmemAccN, "four issuers x two buffers x 32 rows");

// Work split of the narrow kernel.  The unit is a pair block (two k-blocks; the second one of a slab's last pair may lie
// beyond K, where the copies fill zeros).  The (slab, pair block) units are numbered slab-major, total = slabs * pair
// blocks, and CTA c of G takes the contiguous range [total c / G, total (c + 1) / G): every SM streams the same number of
// weight bytes whatever the number of slabs.  A range cuts slabs into segments.  A segment that covers its whole slab is finished by
// its CTA; otherwise the CTA stores its FP32 partial sums as slice (slab, its position among the slab's contributors),
// and the last contributor to arrive (one ticket per slab and epilogue warp) adds the slices in position order - so the
// result does not depend on arrival order - and writes C.
struct NarrowPlan {
    long long total;     // slabs * pair blocks
    float* part;         // [slab][pmax][mp][128] partial sums, or nullptr when every range is made of whole slabs
    unsigned* tickets;   // [slab][4], zero at launch
    int pmax;            // slices per slab
};

// In front of the narrow kernel when the workspace has room: the activations [M,K] (contiguous bytes) expanded to BF16, and
// the status word and the tickets cleared, in one launch.  Its dependents may start at once (the narrow kernel builds its
// table meanwhile and waits for this grid's completion before it reads any of this).
__global__ void __launch_bounds__(256) narrow_prepare_kernel(const uint4* __restrict__ a, uint4* __restrict__ a_bf, unsigned long long n_vec,
                                                             uint32_t* __restrict__ clear, unsigned clear_words)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ uint32_t lut[256];
    lut[threadIdx.x] = hif8_to_bf16_bits(threadIdx.x);
    __syncthreads();
    if (blockIdx.x == 0)
        for (unsigned i = threadIdx.x; i < clear_words; i += 256) clear[i] = 0u;
    for (unsigned long long u = (unsigned long long)blockIdx.x * 256 + threadIdx.x; u < n_vec; u += (unsigned long long)gridDim.x * 256) {
        const uint4 v = a[u];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[8];
#pragma unroll
        for (int i = 0; i < 4; i++) {
            o[2 * i] = lut[w[i] & 0xFFu] | (lut[(w[i] >> 8) & 0xFFu] << 16);
            o[2 * i + 1] = lut[(w[i] >> 16) & 0xFFu] | (lut[w[i] >> 24] << 16);
        }
        a_bf[2 * u] = make_uint4(o[0], o[1], o[2], o[3]);
        a_bf[2 * u + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

template <bool W_IS_NK, bool ACT_BF16>
__global__ void __launch_bounds__(kThreadsN, 1)
hif8_gemm_narrow_kernel(const __grid_constant__ CUtensorMap map_act, const __grid_constant__ CUtensorMap map_w, const GemmParams p, int mp,
                        const NarrowPlan plan)
{
    extern __shared__ unsigned char smem_raw[];
    // the 64 KiB table pays for [N,K] weights, whose bytes are extracted from registers (76 against 85 us at 16 x 28672 x 8192);
    // [K,N] weights arrive a byte per load and ran slower with it (84 against 81 us)
    constexpr bool kWideN = ACT_BF16 && W_IS_NK;
    constexpr int kLutShiftN = kWideN ? 8 : 7;
    const NarrowSmem<kWideN> lay(smem_u32(smem_raw));
    unsigned char* sm = smem_raw - smem_u32(smem_raw);  // generic pointer of shared-window address 0
    {
        uint32_t dyn_bytes;
        asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_bytes));
        if (lay.end > smem_u32(smem_raw) + dyn_bytes) {  // the layout does not fit (the same answer in every thread)
            if (ACT_BF16) asm volatile("griddepcontrol.wait;" ::: "memory");  // (the launch in front clears the status word)
            if (threadIdx.x == 0) atomicCAS(p.status, 0, 7);
            return;
        }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int S = kNwTmemStages;  // operand ring: the it-th k-block uses stage it % S
    static_assert(S % kDecodeGroups == 0, "an operand stage is always written by the same group");
    constexpr int S8 = kNwByteStages;   // byte ring: the i-th pair block of this CTA lands in stage i % S8
    constexpr uint32_t kU8Act = 2 * kNwW8;  // byte stage: 128 weight columns x 128 k, then (activations as bytes) act rows x 128 k
    const uint32_t bars = lay.bars;
    auto bar_u8_full = [&](int s) { return bars + 8u * s; };
    auto bar_u8_empty = [&](int s) { return bars + 8u * (S8 + s); };
    auto bar_bf_full = [&](int s) { return bars + 8u * (2 * S8 + s); };
    auto bar_bf_empty = [&](int s) { return bars + 8u * (2 * S8 + S + s); };
    auto bar_acc_full = [&](int b) { return bars + 8u * (2 * S8 + 2 * S + b); };
    auto bar_acc_empty = [&](int b) { return bars + 8u * (2 * S8 + 2 * S + 2 + b); };
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + lay.abort_flag());
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + lay.tmem_slot());
    uint32_t* lut_all = reinterpret_cast<uint32_t*>(sm + lay.lut);
    const uint32_t lut = lay.lut + 4u * lane;
    const int num_pb = (p.K + BK2 - 1) / BK2, num_kb = 2 * num_pb;  // per slab
    const long long G = gridDim.x;
    const long long pair0 = plan.total * blockIdx.x / G, pair1 = plan.total * (blockIdx.x + 1) / G;  // this CTA's (slab, pair block) range
    const long long lin0 = 2 * pair0, lin1 = 2 * pair1;  // the same in k-blocks
    const int n_pairs = (int)(pair1 - pair0), n_it = 2 * n_pairs;
    const uint32_t act_bytes = (uint32_t)mp * BK2;
    // Up to 32 activation rows: four issuers with two accumulators each (the epilogue of one segment overlaps the next
    // segment's MMAs).  Above that issuers x buffers x rows must stay within 256 columns: four issuers with one accumulator
    // for [N,K] weights (91 against 94 us at 64 x 28672 x 8192), two with two for [K,N] weights (92 against 95 us).
    const int issuers = (mp <= 32 || W_IS_NK) ? kNwMaxIssuers : 2;
    const int bufs = (mp <= 32 || issuers == 2) ? 2 : 1;
    auto acc_col = [&](int q, int buf) { return (uint32_t)((q * bufs + buf) * mp); };  // accumulator of issuer q, buffer buf

    fill_decode_table<(1 << (kLutShiftN - 2))>(lut_all, warp, lane, kThreadsN / 32);  // rows of 1 << kLutShiftN bytes
    if (threadIdx.x == 0) {
        for (int s = 0; s < S8; s++) { mbar_init(bar_u8_full(s), 1); mbar_init(bar_u8_empty(s), 2 * kGroupWarps); }  // both halves' groups
        // operands ready: the group's warps, plus (ACT_BF16) the announcement of the activation tile's bytes
        for (int s = 0; s < S; s++) { mbar_init(bar_bf_full(s), kGroupWarps + (ACT_BF16 ? 1 : 0)); mbar_init(bar_bf_empty(s), 1); }
        for (int b = 0; b < 2; b++) { mbar_init(bar_acc_full(b), issuers); mbar_init(bar_acc_empty(b), kEpiWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(lay.tmem_slot()), "r"(kTmemColsN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The launch in front of this kernel expands the activations and clears the status word and the tickets; this kernel was
    // started while that one ran, so that the set-up above overlaps it.  From here on its results are complete.
    if (ACT_BF16) asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == kTmaWarp) {
        if (lane == 0) {
            int issued = 0, issued_act = 0;
            bool aborted = false;
            const uint64_t w_policy = l2_policy_evict_first();
            int j = (int)(pair0 / num_pb), pb = (int)(pair0 % num_pb);
            for (int it = 0; it < n_pairs; it++) {
                const int s = it % S8, round = it / S8;
                if (round > 0 && !mbar_wait(bar_u8_empty(s), (round - 1) & 1, abort_flag, p.status, 31)) break;
                if (*abort_flag) break;
                const uint32_t dst_w = lay.u8(s), dst_a = dst_w + kU8Act;
                mbar_arrive_expect_tx(bar_u8_full(s), 2 * kNwW8 + (ACT_BF16 ? 0u : act_bytes));
                // (the weight is read once: its lines are the first to leave L2 again, so that the expanded activations, which
                // every CTA reads, and the slices of the slabs that two CTAs share stay there)
                if (W_IS_NK) tma_load_2d_hint(dst_w, &map_w, pb * BK2, j * BM, bar_u8_full(s), w_policy);
                else tma_load_2d_hint(dst_w, &map_w, j * BM, pb * BK2, bar_u8_full(s), w_policy);
                if (!ACT_BF16) tma_load_2d(dst_a, &map_act, pb * BK2, 0, bar_u8_full(s));
                issued = it + 1;
                if (ACT_BF16) {
                    // Activations expanded to BF16 beforehand (map_act is then the map of that copy): the tiles of the pair's
                    // two k-blocks go straight into their operand stages, in the 128-byte-swizzled layout the MMA reads, once
                    // the MMAs of each stage's previous use have read it.  (The byte copy above is needed eight k-blocks later;
                    // these are needed by the end of their k-block's decode, and their waits end about when the next byte
                    // stage falls free, so one thread keeps both streams going.)
                    for (int h = 0; h < 2 && !aborted; h++) {
                        const int ik = 2 * it + h, sb = ik % S, rb = ik / S;
                        if (rb > 0 && !mbar_wait(bar_bf_empty(sb), (rb - 1) & 1, abort_flag, p.status, 37)) { aborted = true; break; }
                        mbar_arrive_expect_tx(bar_bf_full(sb), (uint32_t)mp * BK * 2u);
                        tma_load_2d(lay.bf(sb), &map_act, (2 * pb + h) * BK, 0, bar_bf_full(sb));
                        issued_act = ik + 1;
                    }
                    if (aborted) break;
                }
                if (++pb == num_pb) { pb = 0; j++; }
            }
            if (*abort_flag) {  // let the copies already issued land before this CTA's shared memory goes away
                for (int it = max(0, issued - S8); it < issued; it++) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_u8_full(it % S8), (it / S8) & 1) && global_ns() - t0 < kWaitLimitNs) {}
                }
                for (int ik = max(0, issued_act - S); ik < issued_act; ik++) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_bf_full(ik % S), (ik / S) & 1) && global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == kMmaWarp || warp >= kFirstDecodeWarp + kDecodeWarps) {
        const int q = warp == kMmaWarp ? 0 : warp - (kFirstDecodeWarp + kDecodeWarps) + 1;  // issuer number
        if (lane == 0 && q < issuers) {
            // FP32 accumulator, BF16 operands; A = weight slab (K-major for [N,K] weights, MN-major for [K,N]), B = activations
            // (K-major), N = mp, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(mp >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            // descriptor of stage 0; a stage or a 16-k step further on adds to the address field only
            const uint64_t da0 = make_smem_desc(lay.bf(0), 16, 1024);
            bool ok = true, first = true;
            int kb = (int)(lin0 % num_kb), seg = 0;
            for (int it = 0; it < n_it && ok; it++) {
                const int buf = bufs == 2 ? seg & 1 : 0, use = bufs == 2 ? seg >> 1 : seg;  // use: how often the buffer was filled before
                if ((it & (issuers - 1)) == q) {
                    const int s = it % S, round = it / S;
                    // a segment's first MMA overwrites the accumulator: the epilogue must have read its previous contents
                    if (first && use >= 1) ok = mbar_wait(bar_acc_empty(buf), (use - 1) & 1, abort_flag, p.status, 36);
                    if (ok) ok = mbar_wait(bar_bf_full(s), round & 1, abort_flag, p.status, 32);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc_col(q, buf);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; kk++) {
                        // weights from tensor memory: operand stage s, 16 k = 8 columns
                        tc_mma_bf16_cta_a_tmem(d_tmem, tmem_base + kTmemAccN + (uint32_t)(s * (BK / 2) + kk * 8),
                                               da0 + (uint64_t)((lay.bf(s) - lay.bf(0) + kk * 32) >> 4), idesc, (!first || kk > 0) ? 1u : 0u);
                    }
                    tc_commit_cta(bar_bf_empty(s));
                    first = false;
                }
                if (++kb == num_kb || it == n_it - 1) {  // the segment ends with its slab or with this CTA's range
                    // An issuer without a k-block in the segment only arrives.  With one buffer that arrival must not fall
                    // into the barrier's previous phase (the other issuers' commits of the last segment may still be on
                    // their way): it waits until the epilogue has read the last segment, as a first MMA would have.
                    if (first && bufs == 1 && use >= 1) ok = mbar_wait(bar_acc_empty(buf), (use - 1) & 1, abort_flag, p.status, 36);
                    if (!ok) break;
                    tc_commit_cta(bar_acc_full(buf));
                    kb = 0; seg++; first = true;
                }
            }
        }
    } else if (warp >= kFirstDecodeWarp) {
        const int group = (warp - kFirstDecodeWarp) / kGroupWarps;
        const int dt = threadIdx.x - (kFirstDecodeWarp + group * kGroupWarps) * 32;
        const int act_chunks = mp * (BK / 8);  // 8-byte chunks of the activation tile
        bool ok = true;
        for (int it = group; it < n_it && ok; it += kDecodeGroups) {
            const int s = it % S, r = it / S, s8 = (it >> 1) % S8, h = it & 1;  // h: which k-block of its pair block
            ok = mbar_wait(bar_u8_full(s8), ((it >> 1) / S8) & 1, abort_flag, p.status, 33);
            if (ok && r > 0) ok = mbar_wait(bar_bf_empty(s), (r - 1) & 1, abort_flag, p.status, 34);
            if (!ok) break;
            const uint32_t w8 = lay.u8(s8), a8 = w8 + kU8Act + (uint32_t)h * BK;
            const uint32_t abf = lay.bf(s);
            uint2 va[kNarrowMaxM * (BK / 8) / kGroupThreads];
            uint4 vr[BK / 16];
            // this thread owns weight column (operand row, tensor-memory lane) quarter * 32 + lane of the slab
            const int wr = (warp & 3) * 32 + lane;
            if (W_IS_NK) {
                // [N,K] weights: the byte tile (rows of 128 k) arrives with the 128-byte TMA swizzle (chunk j of row r at chunk
                // j ^ (r & 7)): conflict-free row reads
                const uint32_t w_row = w8 + (uint32_t)wr * BK2, sw = (uint32_t)wr & 7u;
#pragma unroll
                for (int jj = 0; jj < BK / 16; jj++) vr[jj] = lds_v4(w_row + (((uint32_t)(4 * h + jj) ^ sw) << 4));
            }
            if (!ACT_BF16) {
#pragma unroll
                for (int i = 0; i < kNarrowMaxM * (BK / 8) / kGroupThreads; i++) {
                    const int q = i * kGroupThreads + dt;
                    if (q < act_chunks) va[i] = lds_v2(a8 + (q >> 3) * BK2 + (q & 7) * 8);
                }
            }
            uint32_t o[BK / 2];  // 64 BF16 of this weight column, two per tensor-memory column
            if (W_IS_NK) {
                __syncwarp();  // the byte stage has been read: the producer may refill it during the decode
                if (lane == 0) mbar_arrive(bar_u8_empty(s8));
#pragma unroll
                for (int jj = 0; jj < BK / 16; jj++) {
                    const uint4 lo = decode8<kLutShiftN>(make_uint2(vr[jj].x, vr[jj].y), lut), hi = decode8<kLutShiftN>(make_uint2(vr[jj].z, vr[jj].w), lut);
                    o[8 * jj + 0] = lo.x; o[8 * jj + 1] = lo.y; o[8 * jj + 2] = lo.z; o[8 * jj + 3] = lo.w;
                    o[8 * jj + 4] = hi.x; o[8 * jj + 5] = hi.y; o[8 * jj + 6] = hi.z; o[8 * jj + 7] = hi.w;
                }
            } else {
                // [K,N] weights: row k of the pair's tile holds the 128 columns of the slab (the pair's second k-block is its
                // rows 64-127), so the column is read a byte per k: the 32 lanes of a warp read 32 consecutive bytes, one
                // wavefront, and the byte is the table row without any extraction
                const uint32_t w_col = w8 + (uint32_t)h * kNwW8 + (uint32_t)wr;
#pragma unroll
                for (int j = 0; j < BK / 2; j++) {
                    const uint32_t c0 = lds_u8(w_col + (uint32_t)(2 * j) * BM), c1 = lds_u8(w_col + (uint32_t)(2 * j + 1) * BM);
                    // (rows of 256 bytes: the byte replaces byte 1 of the lane's table address, one permute)
                    if (kLutShiftN == 8) o[j] = __byte_perm(lds_u32(__byte_perm(c0, lut, 0x7604)), lds_u32(__byte_perm(c1, lut, 0x7604)), 0x5410);
                    else o[j] = __byte_perm(lds_u32(lut + (c0 << 7)), lds_u32(lut + (c1 << 7)), 0x5410);
                }
                __syncwarp();  // the byte stage has been read
                if (lane == 0) mbar_arrive(bar_u8_empty(s8));
            }
            tmem_st_32x32b_x32(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + kTmemAccN + (uint32_t)(s * (BK / 2)), o);
            if (!ACT_BF16) {
#pragma unroll
                for (int i = 0; i < kNarrowMaxM * (BK / 8) / kGroupThreads; i++) {
                    const int q = i * kGroupThreads + dt, row = q >> 3, jc = q & 7;
                    if (q < act_chunks) sts_v4(abf + (row >> 3) * 1024 + (row & 7) * 128 + ((jc ^ (row & 7)) << 4), decode8<7>(va[i], lut));
                }
            }
            tmem_st_wait();  // the weight column is in tensor memory
            if (!ACT_BF16) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_bf_full(s));
        }
    } else {
        // epilogue warps 0-3: TMEM lane = weight column n, TMEM column = activation row m
        const int sa = p.d_sa ? *p.d_sa : 0;
        long long lin = lin0;
        for (int seg = 0; lin < lin1; seg++) {
            const int j = (int)(lin / num_kb), kb_a = (int)(lin % num_kb), buf = bufs == 2 ? seg & 1 : 0, use = bufs == 2 ? seg >> 1 : seg;
            const long long slab_end = (long long)(j + 1) * num_kb, seg_end = slab_end < lin1 ? slab_end : lin1;
            const bool whole = kb_a == 0 && seg_end == slab_end;
            if (!mbar_wait(bar_acc_full(buf), use & 1, abort_flag, p.status, 35)) break;
            tc_fence_after();
            const int n = j * BM + warp * 32 + lane;
            const int sw = p.d_sw_channel ? (n < p.N ? p.d_sw_channel[n] : 0) : (p.d_sw ? *p.d_sw : 0);
            const int sc = -(sa + sw), s1 = sc / 2, s2 = sc - s1;
            const float f1 = __uint_as_float((uint32_t)(s1 + 127) << 23), f2 = __uint_as_float((uint32_t)(s2 + 127) << 23);
            auto finish = [&](int m, float acc) {  // C[m][n] from the complete sum
                float v = acc * f1 * f2;
                if (p.c_is_f32) {
                    float* out = reinterpret_cast<float*>(p.C) + (long long)m * p.ldc + n;
                    *out = p.accumulate ? v + *out : v;
                } else {
                    unsigned short* out = reinterpret_cast<unsigned short*>(p.C) + (long long)m * p.ldc + n;
                    if (p.accumulate) v += __uint_as_float((uint32_t)*out << 16);
                    unsigned short b;
                    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(b) : "f"(v));  // round to nearest even; a NaN stays a NaN
                    *out = b;
                }
            };
            // contributors of slab j are the CTAs owner(first pair block) .. owner(last pair block);
            // owner(x) = the largest c with total c / G <= x
            const long long c_first = (((long long)j * num_pb + 1) * G - 1) / plan.total, c_last = ((long long)(j + 1) * num_pb * G - 1) / plan.total;
            const int pos = (int)(blockIdx.x - c_first), count = (int)(c_last - c_first + 1);
            float* slab_part = whole ? nullptr : plan.part + (size_t)j * plan.pmax * mp * BM + warp * 32 + lane;
            float* mine = whole ? nullptr : slab_part + (size_t)pos * mp * BM;
            const uint32_t tlane = tmem_base + ((uint32_t)(warp * 32) << 16);
            const int it_a = (int)(lin - lin0), it_n = (int)(seg_end - lin);  // the segment's k-blocks, counted within this CTA's range
            for (int c = 0; c < mp; c += 32) {
                float r[32];  // this lane's row of the segment's sum, columns c .. c + 31: the issuers' accumulators added in order
#pragma unroll
                for (int i = 0; i < 32; i++) r[i] = 0.f;
                for (int q = 0; q < issuers; q++) {
                    // issuer q took the k-blocks it = q (mod issuers): none of them in a short segment leaves its accumulator stale
                    if (it_n < issuers && ((q - it_a) & (issuers - 1)) >= it_n) continue;
                    uint32_t t[32];
                    tmem_ld_32x32b_x32(tlane + acc_col(q, buf) + c, t);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; i++) r[i] += __uint_as_float(t[i]);
                }
                if (whole) {
                    if (n < p.N) {
#pragma unroll
                        for (int i = 0; i < 32; i++)
                            if (c + i < p.M) finish(c + i, r[i]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i++)
                        if (c + i < mp) __stcg(mine + (c + i) * BM, r[i]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty(buf));  // the accumulator has been read: it may be overwritten
            if (!whole) {
                __threadfence();
                __syncwarp();
                unsigned prior = 0;
                if (lane == 0) prior = atomicAdd(plan.tickets + j * kEpiWarps + warp, 1u);
                prior = __shfl_sync(0xFFFFFFFFu, prior, 0);
                if (prior == (unsigned)(count - 1)) {  // every slice of this quarter slab is complete
                    __threadfence();
                    if (n < p.N) {
                        // sixteen rows at a time: their loads are independent, so the L2 latency is paid once per slice
                        for (int m0 = 0; m0 < p.M; m0 += 16) {
                            float acc[16];
                            if (count == 2) {
                                // two contributors (the usual case): both slices' loads in flight together, same order of addition
                                float v0[16], v1[16];
#pragma unroll
                                for (int u = 0; u < 16; u++) v0[u] = __ldcg(slab_part + (size_t)m0 * BM + u * BM);
#pragma unroll
                                for (int u = 0; u < 16; u++) v1[u] = __ldcg(slab_part + ((size_t)mp + m0) * BM + u * BM);
#pragma unroll
                                for (int u = 0; u < 16; u++)
                                    if (m0 + u < p.M) finish(m0 + u, (0.f + v0[u]) + v1[u]);
                                continue;
                            }
#pragma unroll
                            for (int u = 0; u < 16; u++) acc[u] = 0.f;
                            for (int i = 0; i < count; i++) {
                                const float* sl = slab_part + ((size_t)i * mp + m0) * BM;  // m0 + 15 < mp: mp is a multiple of 16
                                float v[16];
#pragma unroll
                                for (int u = 0; u < 16; u++) v[u] = __ldcg(sl + u * BM);
#pragma unroll
                                for (int u = 0; u < 16; u++) acc[u] += v[u];
                            }
#pragma unroll
                            for (int u = 0; u < 16; u++)
                                if (m0 + u < p.M) finish(m0 + u, acc[u]);
                        }
                    }
                }
            }
            lin = seg_end;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemColsN) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------------------
// Decode-once path: operands already decoded to BF16 (by the conversion kernels of this library, into the caller's
// workspace).  Persistent kernel on CTA pairs (cta_group::2), 64-wide k-blocks.
//   warps 0-3  epilogue (TMEM -> global), overlapped with the next tile through two TMEM accumulators
//   warp  4    TMA producer of the A tiles: BF16 tiles land directly in the 128-byte-swizzled operand layout
//   warp  5    MMA issuer
//   warp  6    TMA producer of the W tiles (issuing a tile copy costs its thread about 200 cycles; one thread issuing the
//              two or three copies of a k-block, with its waits, took longer than the 512 cycles of the k-block's MMAs)
// A cluster of two CTAs on two SMs computes one 256 x 256 tile: each CTA stages its own 128 rows of A and its own 128
// columns of W (so the tensor core reads half as many operand bytes per SM and flop as with one CTA per tile, which is
// what bounds a one-CTA kernel), both accumulate their 128 rows in their own TMEM.  The even CTA of the pair (the
// leader) issues every tcgen05.mma; its commits arrive on the barriers of both CTAs.  TMA copies of both CTAs complete
// on the leader's "full" barrier (no multicast loads).
// ---------------------------------------------------------------------------------------------------------
constexpr int kThreadsP = 7 * 32;
constexpr int kTmaWarpW = 6;
constexpr int kStages2 = 6;
constexpr uint32_t kStageBytes2 = kABfBytes + kBBfBytes;            // 32 KiB per CTA and stage
struct SmemLayout2 {
    static constexpr uint32_t bars = kStages2 * kStageBytes2;         // 192 KiB
    static constexpr uint32_t n_bars = 2 * kStages2 + 4;
    static constexpr uint32_t tmem_slot = bars + n_bars * 8;
    static constexpr uint32_t abort_flag = tmem_slot + 4;
    static constexpr uint32_t total = abort_flag + 4;
};
constexpr uint32_t kSmemBytes2 = SmemLayout2::total + 1024;

template <bool W_IS_NK>
__global__ void __launch_bounds__(kThreadsP, 1)
bf16_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const GemmParams p)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0: leader (issues the MMAs), 1: peer
    const bool leader = rank == 0;
    const uint32_t bars = base + SmemLayout2::bars;
    auto bar_full = [&](int s) { return bars + 8u * s; };                       // used in the leader only
    auto bar_empty = [&](int s) { return bars + 8u * (kStages2 + s); };         // per CTA, released by the leader's commits
    auto bar_acc_full = [&](int a) { return bars + 8u * (2 * kStages2 + a); };  // per CTA
    auto bar_acc_empty = [&](int a) { return bars + 8u * (2 * kStages2 + 2 + a); };  // leader: both epilogues arrive
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + SmemLayout2::abort_flag);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + SmemLayout2::tmem_slot);
    const int num_kb = (p.K + BK - 1) / BK;
    const int tiles_m2 = (p.M + 2 * BM - 1) / (2 * BM), tiles_n2 = p.tiles_n;
    // a batch of n x n products (A variant ia, W variant iw) is one list of tiles: product b = ia * n + iw owns tiles
    // [b * tiles_one, (b + 1) * tiles_one)
    const int tiles_one = tiles_m2 * tiles_n2, nb = p.batch_n > 0 ? p.batch_n : 1;
    const int tiles = tiles_one * nb * nb, pairs = gridDim.x >> 1, pair_id = blockIdx.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages2; s++) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int a = 0; a < 2; a++) { mbar_init(bar_acc_full(a), 1); mbar_init(bar_acc_empty(a), 2 * kEpiWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + SmemLayout2::tmem_slot), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // barriers of both CTAs are initialised before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == kTmaWarp || warp == kTmaWarpW) {
        if (lane == 0) {
            const bool loads_a = warp == kTmaWarp;
            long long issued = 0;
            int s = 0;            // stage of the next k-block
            uint32_t ph = 0;      // parity of the round the ring is in
            bool ok = true, wrapped = false;
            for (int t = pair_id; t < tiles && ok; t += pairs) {
                int tile_m, tile_n;
                const int b = t / tiles_one, ia = b / nb, iw = b - ia * nb;
                tile_coords(t - b * tiles_one, tiles_m2, tiles_n2, tile_m, tile_n);
                const int m0 = tile_m * 2 * BM + (int)rank * BM, n0 = tile_n * BN + (int)rank * (BN / 2);
                for (int kb = 0; kb < num_kb; kb++) {
                    if (wrapped) ok = mbar_wait(bar_empty(s), ph ^ 1u, abort_flag, p.status, 21);  // the previous round's use of the stage
                    if (!ok || *abort_flag) { ok = false; break; }
                    const uint32_t dst_a = base + s * kStageBytes2, dst_b = dst_a + kABfBytes;
                    const uint32_t full = map_to_cta(bar_full(s), 0);
                    if (loads_a) {
                        if (leader) mbar_arrive_expect_tx(bar_full(s), 2 * kStageBytes2);  // bytes of both CTAs, both operands
                        tma_load_3d_pair(dst_a, &map_a, kb * BK, m0, ia, full);
                    } else if (W_IS_NK) tma_load_3d_pair(dst_b, &map_w, kb * BK, n0, iw, full);
                    else {
#pragma unroll
                        for (int c = 0; c < BN / 2 / 64; c++)
                            tma_load_3d_pair(dst_b + c * 8192, &map_w, n0 + c * 64, kb * BK, iw, full);
                    }
                    issued++;
                    if (++s == kStages2) { s = 0; ph ^= 1u; wrapped = true; }
                }
            }
            if (*abort_flag && leader && loads_a) {  // let copies in flight land (their completions are counted on the leader)
                for (long long j = issued > kStages2 ? issued - kStages2 : 0; j < issued; j++) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full((int)(j % kStages2)), (uint32_t)((j / kStages2) & 1)) &&
                           global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == kMmaWarp) {
        if (lane == 0 && leader) {
            // M = 256 over the pair, N = 256
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((W_IS_NK ? 0u : 1u) << 16) |
                                   ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
            int local = 0, s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int t = pair_id; t < tiles && ok; t += pairs, local++) {
                const int acc = local & 1, use = local >> 1;
                if (use > 0) ok = mbar_wait(bar_acc_empty(acc), (uint32_t)((use - 1) & 1), abort_flag, p.status, 22);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * 256;
                for (int kb = 0; kb < num_kb; kb++) {
                    ok = mbar_wait(bar_full(s), ph, abort_flag, p.status, 23);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = base + s * kStageBytes2, b_addr = a_addr + kABfBytes;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; kk++) {
                        const uint64_t da = make_smem_desc(a_addr + kk * 32, 16, 1024);
                        const uint64_t db = W_IS_NK ? make_smem_desc(b_addr + kk * 32, 16, 1024)
                                                    : make_smem_desc(b_addr + kk * 2048, 8192, 1024);
                        tc_mma_bf16_pair(d_tmem, da, db, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit_pair(bar_empty(s));
                    if (++s == kStages2) { s = 0; ph ^= 1u; }
                }
                if (ok) tc_commit_pair(bar_acc_full(acc));
            }
        }
    } else if (warp < kEpiWarps) {
        int local = 0, b_held = -1;
        double err_acc = 0.0;  // squared-error variant: this thread's share of product b_held
        const bool ref_vec = !(reinterpret_cast<uintptr_t>(p.err_ref) & 15) && !(p.ld_ref & 3);
        auto flush_error = [&]() {  // all lanes of the warp
            for (int off = 16; off > 0; off >>= 1) err_acc += __shfl_xor_sync(0xFFFFFFFFu, err_acc, off);
            if (lane == 0 && err_acc != 0.0 && b_held >= 0) atomicAdd(p.err_sum + b_held, err_acc);
            err_acc = 0.0;
        };
        for (int t = pair_id; t < tiles; t += pairs, local++) {
            const int acc = local & 1, use = local >> 1;
            if (!mbar_wait(bar_acc_full(acc), (uint32_t)(use & 1), abort_flag, p.status, 24)) break;
            tc_fence_after();
            int tile_m, tile_n;
            const int b = t / tiles_one, ia = b / nb, iw = b - ia * nb;
            if (p.err_sum && b != b_held) { flush_error(); b_held = b; }
            // exponents of this product (in a batch: entry ia / iw of the two device arrays)
            const int sa = p.d_sa ? p.d_sa[ia] : 0;
            const int sdesc = p.d_sw_channel ? 0 : -(sa + (p.d_sw ? p.d_sw[iw] : 0));
            const int s1 = sdesc / 2, s2 = sdesc - s1;
            const float f1 = __uint_as_float((uint32_t)(s1 + 127) << 23), f2 = __uint_as_float((uint32_t)(s2 + 127) << 23);
            tile_coords(t - b * tiles_one, tiles_m2, tiles_n2, tile_m, tile_n);
            const int row = tile_m * 2 * BM + (int)rank * BM + warp * 32 + lane, n0 = tile_n * BN;
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(warp * 32) << 16) + acc * 256 + c, r);
                tmem_ld_wait();
                const int col = n0 + c;
                if (p.d_sw_channel) apply_channel_scale(p, col, lane, sa, r);
                if (p.err_sum) {
                    if (row < p.M && col < p.N) {
                        // exact differences of the FP32 result and the FP32 reference, squared and summed in double
                        const float* ref = p.err_ref + (long long)row * p.ld_ref + col;
                        if (col + 32 <= p.N && ref_vec) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4) {
                                const float4 o = __ldg(reinterpret_cast<const float4*>(ref + i));
                                const double d0 = (double)(__uint_as_float(r[i]) * f1 * f2) - (double)o.x;
                                const double d1 = (double)(__uint_as_float(r[i + 1]) * f1 * f2) - (double)o.y;
                                const double d2 = (double)(__uint_as_float(r[i + 2]) * f1 * f2) - (double)o.z;
                                const double d3 = (double)(__uint_as_float(r[i + 3]) * f1 * f2) - (double)o.w;
                                err_acc += d0 * d0 + d1 * d1 + d2 * d2 + d3 * d3;
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; i++) {  // (constant indices: see store_chunk)
                                if (col + i < p.N) {
                                    const double d = (double)(__uint_as_float(r[i]) * f1 * f2) - (double)__ldg(ref + i);
                                    err_acc += d * d;
                                }
                            }
                        }
                    }
                } else store_chunk(p, row, col, r, f1, f2);
            }
            tc_fence_before();
            __syncwarp();
            // (default semantics: what the leader's MMAs must not overtake are this warp's tensor-memory loads, ordered by
            // tcgen05.wait::ld and the fence above -- not its stores to C, which a release at cluster scope would wait for)
            if (lane == 0) mbar_arrive_remote(map_to_cta(bar_acc_empty(acc), 0));  // tell the leader: accumulator drained
        }
        if (p.err_sum) flush_error();
    }

    // nobody leaves while the other CTA may still read this CTA's shared memory or signal its barriers
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing will ever complete, with a short limit.
// The wait must give up, record its status word and let the kernel finish normally.
__global__ void wait_selftest_kernel(int* status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) (void)mbar_wait(smem_u32(&bar), 0, &abort_flag, status, 99, limit_ns);
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

// Tensor maps are cached per (pointer, shape, leading dimension, box): encoding one costs a driver call of a few
// microseconds, which matters for the narrow products of ~100 us when the same operands come back call after call.
struct MapKey {
    const void* ptr;
    uint64_t inner, rows, count, ld;  // ld: row pitch in elements (2-D) or distance between stacked matrices (3-D)
    uint32_t box_inner, box_rows;
    uint32_t kind;                    // 0: bytes, 2-D; 1: BF16, 2-D, 128-byte swizzle; 2: BF16, 3-D stack, 128-byte swizzle;
                                      // 3: bytes, 2-D, 64-byte swizzle; 4: bytes, 2-D, 128-byte swizzle
    uint32_t pad;
};
LruCache<MapKey, CUtensorMap, 64> g_map_cache;

bool encode_map(const MapKey& k, CUtensorMap* map)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const bool bf16 = k.kind == 1 || k.kind == 2;
    if (k.kind == 2) {
        cuuint64_t dims[3] = {k.inner, k.rows, k.count};
        cuuint64_t strides[2] = {k.inner * 2u, (k.count > 1 ? k.ld : k.inner * k.rows) * 2u};
        cuuint32_t box[3] = {k.box_inner, k.box_rows, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(k.ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    cuuint64_t dims[2] = {k.inner, k.rows};
    cuuint64_t strides[1] = {k.ld * (bf16 ? 2u : 1u)};
    cuuint32_t box[2] = {k.box_inner, k.box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(k.ptr), dims,
              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              (bf16 || k.kind == 4) ? CU_TENSOR_MAP_SWIZZLE_128B : (k.kind == 3 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE),
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D tensor [rows][ld elements] with a box of box_inner x box_rows elements, zero fill out of bounds.
// bf16 = false: bytes, with no swizzle or the 64- or 128-byte one (box_inner at most that many bytes).  bf16 = true: 16-bit
// elements, 128-byte swizzle (box_inner must be 64).
bool make_map(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t rows, uint64_t ld, uint32_t box_inner, uint32_t box_rows,
              bool bf16 = false, uint32_t bytes_swizzle = 0)
{
    MapKey k;
    std::memset(&k, 0, sizeof k);
    k.ptr = ptr; k.inner = inner; k.rows = rows; k.count = 1; k.ld = ld; k.box_inner = box_inner; k.box_rows = box_rows;
    k.kind = bf16 ? 1u : (bytes_swizzle == 64 ? 3u : (bytes_swizzle == 128 ? 4u : 0u));
    return g_map_cache.lookup_or_make(k, map, encode_map);
}

// BF16 stack of `count` matrices [rows, inner], `stack_stride` elements apart (box: one matrix deep)
bool make_map3(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t rows, uint64_t count, uint64_t stack_stride,
               uint32_t box_inner, uint32_t box_rows)
{
    MapKey k;
    std::memset(&k, 0, sizeof k);
    k.ptr = ptr; k.inner = inner; k.rows = rows; k.count = count; k.ld = count > 1 ? stack_stride : 0; k.box_inner = box_inner;
    k.box_rows = box_rows; k.kind = 2u;
    return g_map_cache.lookup_or_make(k, map, encode_map);
}

// Kernel attributes (opt-in to more than 48 KiB of dynamic shared memory) and the SM count are facts of one device:
// they are set up once per device ordinal, by the first GEMM call made with that device current.
struct GemmDeviceSetup {
    cudaError_t rc;
    int sm_count;
};
PerDevice<GemmDeviceSetup> g_gemm_setup;

bool gemm_kernels_ready(int dev, int* sm_count_out)
{
    const GemmDeviceSetup* s = g_gemm_setup.get(dev, [](int d, GemmDeviceSetup* out) {
        out->rc = cudaSuccess;
        out->sm_count = 0;
        if (out->rc == cudaSuccess)
            out->rc = cudaFuncSetAttribute(hif8_gemm_kernel<0, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytesSwapped);
        const void* fused[6] = {(const void*)hif8_gemm_kernel<0, false>, (const void*)hif8_gemm_kernel<0, true>,
                                (const void*)hif8_gemm_kernel<1, false>, (const void*)hif8_gemm_kernel<1, true>,
                                (const void*)hif8_gemm_kernel<2, false>, (const void*)hif8_gemm_kernel<2, true>};
        const void* pair[2] = {(const void*)bf16_gemm_pair_kernel<false>, (const void*)bf16_gemm_pair_kernel<true>};
        for (int i = 0; i < 6 && out->rc == cudaSuccess; i++)  // [M,K] byte activations (the first two): the wide-table plan
            out->rc = cudaFuncSetAttribute(fused[i], cudaFuncAttributeMaxDynamicSharedMemorySize, i < 2 ? kSmemBytesWide : kSmemBytes);
        for (int i = 0; i < 2 && out->rc == cudaSuccess; i++)
            out->rc = cudaFuncSetAttribute(pair[i], cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2);
        const void* narrow[4] = {(const void*)hif8_gemm_narrow_kernel<false, false>, (const void*)hif8_gemm_narrow_kernel<false, true>,
                                 (const void*)hif8_gemm_narrow_kernel<true, false>, (const void*)hif8_gemm_narrow_kernel<true, true>};
        for (int i = 0; i < 4 && out->rc == cudaSuccess; i++)
            out->rc = cudaFuncSetAttribute(narrow[i], cudaFuncAttributeMaxDynamicSharedMemorySize, i == 3 ? kSmemBytesWide : kSmemBytesN);  // (the last one: wide table)
        if (out->rc == cudaSuccess) out->rc = cudaDeviceGetAttribute(&out->sm_count, cudaDevAttrMultiProcessorCount, d);
    });
    if (!s) return false;
    *sm_count_out = s->sm_count;
    return s->rc == cudaSuccess && s->sm_count > 0;
}

// The status word of the most recent GEMM-class call per stream, for hif8_last_device_status.
struct StatusKey {
    const void* stream;
};
struct StatusVal {
    const int* word;
    int dev;
};
LruCache<StatusKey, StatusVal, 64> g_last_status;

constexpr size_t kGemmWorkspaceBytes = 256;

}  // namespace

void note_status_word(cudaStream_t st, const int* word)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return;
    StatusKey k;
    std::memset(&k, 0, sizeof k);
    k.stream = st;
    g_last_status.put(k, StatusVal{word, dev});
}

int launch_bf16_pair_gemm(const void* a_bf, const void* w_bf, int w_is_nk, GemmParams p, cudaStream_t st,
                          long long a_stack_stride, long long w_stack_stride)
{
    int dev = 0, sm_count = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || !gemm_kernels_ready(dev, &sm_count)) return HIF8_ERR_CUDA;
    const int M = p.M, N = p.N, K = p.K;
    const uint64_t nb = p.batch_n > 0 ? (uint64_t)p.batch_n : 1;
    p.tiles_m = (M + BM - 1) / BM;
    p.tiles_n = (N + BN - 1) / BN;
    const long long tiles2 = (long long)((M + 2 * BM - 1) / (2 * BM)) * p.tiles_n * (long long)(nb * nb);
    if (M <= 0 || N <= 0 || K <= 0 || tiles2 > 0x3FFFFFFF) return HIF8_ERR_SHAPE;
    if (nb > 1 && ((a_stack_stride & 7) || (w_stack_stride & 7))) return HIF8_ERR_ALIGN;  // 16-byte strides
    CUtensorMap ma, mw;
    // A boxes: this CTA's 128 rows of [M,K]
    if (!make_map3(&ma, a_bf, (uint64_t)K, (uint64_t)M, nb, (uint64_t)a_stack_stride, BK, BM)) return HIF8_ERR_CUDA;
    // W boxes are one CTA's half of the 256-column tile: 128 rows of [N,K], or two boxes of 64 columns of [K,N]
    const bool okw = w_is_nk ? make_map3(&mw, w_bf, (uint64_t)K, (uint64_t)N, nb, (uint64_t)w_stack_stride, BK, BN / 2)
                             : make_map3(&mw, w_bf, (uint64_t)N, (uint64_t)K, nb, (uint64_t)w_stack_stride, 64, BK);
    if (!okw) return HIF8_ERR_CUDA;
    const int pairs = (int)(tiles2 < sm_count / 2 ? tiles2 : sm_count / 2);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2u * (unsigned)pairs);
    cfg.blockDim = dim3(kThreadsP);
    cfg.dynamicSmemBytes = kSmemBytes2;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t lrc = w_is_nk ? cudaLaunchKernelEx(&cfg, bf16_gemm_pair_kernel<true>, ma, mw, p)
                                    : cudaLaunchKernelEx(&cfg, bf16_gemm_pair_kernel<false>, ma, mw, p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return (lrc == cudaSuccess && cudaGetLastError() == cudaSuccess) ? HIF8_OK : HIF8_ERR_CUDA;
}

}  // namespace hif8

using namespace hif8;

static std::atomic<int> g_path_policy{HIF8_GEMM_PATH_AUTO};

extern "C" int hif8_gemm_path_policy(int policy)
{
    if (policy != HIF8_GEMM_PATH_AUTO && policy != HIF8_GEMM_PATH_EXPAND_BOTH) return HIF8_ERR_FLAGS;
    return g_path_policy.exchange(policy, std::memory_order_relaxed);
}

static int gemm_entry(const uint8_t* Aq, int64_t lda, int a_is_km, const uint8_t* Wq, int64_t ldw, int w_is_nk, void* C,
                      int64_t ldc, int c_dtype, int M, int N, int K, const int* d_scale_exp_a, const int* d_scale_exp_w,
                      const int* d_scale_exp_w_channel, int accumulate, void* workspace, size_t workspace_bytes,
                      hif8_stream_t stream)
{
    if (c_dtype != HIF8_BF16 && c_dtype != HIF8_F32) return HIF8_ERR_DTYPE;
    if (M < 0 || N < 0 || K < 0 || (K & 15)) return HIF8_ERR_SHAPE;
    if (lda < (a_is_km ? M : K) || ldc < N || ldw < (w_is_nk ? K : N)) return HIF8_ERR_SHAPE;
    if (M == 0 || N == 0) return HIF8_OK;
    if (!Aq || !Wq || !C) return HIF8_ERR_NULL;
    const size_t c_item = c_dtype == HIF8_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(Aq) & 15) || (reinterpret_cast<uintptr_t>(Wq) & 15) || (reinterpret_cast<uintptr_t>(C) & 15) ||
        (lda & 15) || (ldw & 15) || ((ldc * c_item) & 15))
        return HIF8_ERR_ALIGN;
    if (!workspace || workspace_bytes < kGemmWorkspaceBytes || (reinterpret_cast<uintptr_t>(workspace) & 15))
        return HIF8_ERR_WORKSPACE;
    if (K == 0) return HIF8_ERR_SHAPE;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return HIF8_ERR_CUDA;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (major != 10) return HIF8_ERR_CUDA;

    CUtensorMap map_a, map_w;
    // ([M,K] activations: 64-byte rows with the 64-byte swizzle, read row-wise by the decode warps of the fused kernel)
    const bool ok_a = a_is_km ? make_map(&map_a, Aq, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BM, BK)
                              : make_map(&map_a, Aq, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK, BM, false, 64);
    if (!ok_a) return HIF8_ERR_CUDA;
    // byte tiles of one CTA of a pair: 128 rows of A, 128 of the 256 columns of W
    const bool ok_w = w_is_nk ? make_map(&map_w, Wq, (uint64_t)K, (uint64_t)N, (uint64_t)ldw, BK, BN / 2)
                              : make_map(&map_w, Wq, (uint64_t)N, (uint64_t)K, (uint64_t)ldw, BN / 2, BK);
    if (!ok_w) return HIF8_ERR_CUDA;

    GemmParams p{};
    p.C = C; p.ldc = ldc; p.c_is_f32 = c_dtype == HIF8_F32; p.M = M; p.N = N; p.K = K;
    p.d_sa = d_scale_exp_a; p.d_sw = d_scale_exp_w; p.d_sw_channel = d_scale_exp_w_channel;
    p.accumulate = accumulate ? 1 : 0;
    p.status = reinterpret_cast<int*>(workspace);
    p.tiles_m = (M + BM - 1) / BM; p.tiles_n = (N + BN - 1) / BN;
    // both kernels work on 256 x 256 tiles, one per pair of CTAs
    const long long tiles2 = (long long)((M + 2 * BM - 1) / (2 * BM)) * p.tiles_n;
    if (tiles2 > 0x3FFFFFFF) return HIF8_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    note_status_word(st, reinterpret_cast<const int*>(workspace));

    int sm_count = 0;
    if (!gemm_kernels_ready(dev, &sm_count)) return HIF8_ERR_CUDA;
    // the status word is cleared on the stream before the kernels; the narrow path clears its tickets in the same operation
    size_t clear_bytes = 4;

    // Narrow products: the weight-streaming kernel, whatever the workspace
    if (!a_is_km && M <= kNarrowMaxM) {
        const int mp = (M + 15) & ~15;
        CUtensorMap map_act, map_ws;
        if (!make_map(&map_act, Aq, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK2, (uint32_t)mp)) return HIF8_ERR_CUDA;
        // ([N,K] weights: 64-byte rows with the 64-byte swizzle, read row-wise and decoded into tensor memory)
        const bool okn = w_is_nk ? make_map(&map_ws, Wq, (uint64_t)K, (uint64_t)N, (uint64_t)ldw, BK2, BM, false, 128)
                                 : make_map(&map_ws, Wq, (uint64_t)N, (uint64_t)K, (uint64_t)ldw, BM, BK2);
        if (!okn) return HIF8_ERR_CUDA;
        const long long slabs = (N + BM - 1) / BM, num_pb = (K + BK2 - 1) / BK2;  // pair blocks: two k-blocks
        NarrowPlan plan{};
        plan.total = slabs * num_pb;
        // One CTA per SM, equal k-block ranges, when the workspace holds the partial sums of the slabs that a range
        // boundary cuts; otherwise one CTA per slab.
        long long grid = slabs;
        {
            // aim at four or more pair blocks per CTA, but never fewer CTAs than the per-slab grid would keep busy
            long long g = plan.total / 4 < sm_count ? plan.total / 4 : sm_count;
            const long long floor_g = slabs < sm_count ? slabs : sm_count;
            if (g < floor_g) g = floor_g;
            const long long per = plan.total / g;
            const long long pmax = (num_pb + per - 1) / per + 1;
            const size_t ticket_bytes = (((size_t)slabs * kEpiWarps * 4) + 255) & ~(size_t)255;
            const size_t part_bytes = (size_t)slabs * pmax * mp * BM * 4;
            if (g != slabs && workspace_bytes >= kGemmWorkspaceBytes + ticket_bytes + part_bytes && !(reinterpret_cast<uintptr_t>(workspace) & 255)) {
                unsigned char* wsb = reinterpret_cast<unsigned char*>(workspace) + kGemmWorkspaceBytes;
                plan.tickets = reinterpret_cast<unsigned*>(wsb);
                plan.part = reinterpret_cast<float*>(wsb + ticket_bytes);
                plan.pmax = (int)pmax;
                grid = g;
                clear_bytes = kGemmWorkspaceBytes + ticket_bytes;  // the tickets follow the status block
            }
        }
        if (grid > 0x7FFFFFFFll) return HIF8_ERR_SHAPE;
        // With room left for the activations as BF16 (2 M K bytes behind the partial sums) they are expanded once, here,
        // and their tiles are copied straight into the operand stages: otherwise every CTA decodes the activation tile of
        // every k-block again for each of its slabs, a seventh (16 rows) to a third (64 rows) of the kernel's table lookups.
        bool act_bf16 = false;
        {
            const size_t used = clear_bytes > 4 ? clear_bytes + (size_t)slabs * plan.pmax * mp * BM * 4 : kGemmWorkspaceBytes;
            const size_t off = (used + 255) & ~(size_t)255, bytes_act = (size_t)M * K * 2;
            if (lda == K && workspace_bytes >= off + bytes_act && !(reinterpret_cast<uintptr_t>(workspace) & 255)) {
                unsigned char* a_bf = reinterpret_cast<unsigned char*>(workspace) + off;
                if (!make_map(&map_act, a_bf, (uint64_t)K, (uint64_t)M, (uint64_t)K, BK, (uint32_t)mp, true)) return HIF8_ERR_CUDA;
                const unsigned long long n_vec = (unsigned long long)M * K / 16;  // K is a multiple of 16
                const unsigned long long want = (n_vec + 255) / 256, cap = (unsigned long long)sm_count * 4;
                narrow_prepare_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(
                    reinterpret_cast<const uint4*>(Aq), reinterpret_cast<uint4*>(a_bf), n_vec, reinterpret_cast<uint32_t*>(workspace),
                    (unsigned)(clear_bytes / 4));
                if (cudaGetLastError() != cudaSuccess) return HIF8_ERR_CUDA;
                g_launches.fetch_add(1, std::memory_order_relaxed);
                act_bf16 = true;
            }
        }
        if (!act_bf16 && cudaMemsetAsync(workspace, 0, clear_bytes, st) != cudaSuccess) return HIF8_ERR_CUDA;
        cudaLaunchConfig_t cn{};
        cn.gridDim = dim3((unsigned)grid);
        cn.blockDim = dim3(kThreadsN);
        cn.dynamicSmemBytes = (act_bf16 && w_is_nk) ? kSmemBytesWide : kSmemBytesN;
        cn.stream = st;
        // with the preparing kernel right in front: programmatic stream serialization (that kernel lets its dependents start
        // at once; this one waits for its completion once its own set-up is done)
        cudaLaunchAttribute an[1];
        an[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        an[0].val.programmaticStreamSerializationAllowed = 1;
        cn.attrs = an; cn.numAttrs = act_bf16 ? 1 : 0;
        cudaError_t nrc;
        if (w_is_nk) nrc = act_bf16 ? cudaLaunchKernelEx(&cn, hif8_gemm_narrow_kernel<true, true>, map_act, map_ws, p, mp, plan)
                                    : cudaLaunchKernelEx(&cn, hif8_gemm_narrow_kernel<true, false>, map_act, map_ws, p, mp, plan);
        else nrc = act_bf16 ? cudaLaunchKernelEx(&cn, hif8_gemm_narrow_kernel<false, true>, map_act, map_ws, p, mp, plan)
                            : cudaLaunchKernelEx(&cn, hif8_gemm_narrow_kernel<false, false>, map_act, map_ws, p, mp, plan);
        if (nrc != cudaSuccess) return HIF8_ERR_CUDA;
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
    }

    if (cudaMemsetAsync(workspace, 0, clear_bytes, st) != cudaSuccess) return HIF8_ERR_CUDA;
    // Decode-once path: with room for both operands as BF16 in the workspace (and contiguous operands), each HiF8
    // byte is decoded exactly once by the conversion kernel and the tensor-core kernel reads BF16 tiles through TMA.
    // Otherwise the fused kernel decodes the byte tiles of every CTA in shared memory.
    const size_t bytes_a = (((size_t)M * K * 2) + 255) & ~(size_t)255, bytes_w = (((size_t)K * N * 2) + 255) & ~(size_t)255;
    const bool contiguous = lda == (a_is_km ? M : K) && ldw == (w_is_nk ? K : N);
    // Expanding W as well only pays when the product is large enough to win back the pass over W (3 bytes per element
    // moved) at the higher rate of the decode-once kernel: with about 268 flops per byte of copy bandwidth for that kernel,
    // 233 for the swapped A-expanded form ([N,K] weights) and 210 for the other (their measured rates against the copy rate)
    // they meet near M = 4800 and M = 1450, whatever N and K.
    const double mk = (double)M * K, kn = (double)K * N, flops = 2.0 * mk * N;
    const bool w_expansion_pays = g_path_policy.load(std::memory_order_relaxed) == HIF8_GEMM_PATH_EXPAND_BOTH ||
                                  3.0 * kn + flops / 268.0 < flops / (w_is_nk ? 233.0 : 210.0);
    if (contiguous && w_expansion_pays && workspace_bytes >= kGemmWorkspaceBytes + bytes_a + bytes_w &&
        !(reinterpret_cast<uintptr_t>(workspace) & 255)) {
        unsigned char* a_bf = reinterpret_cast<unsigned char*>(workspace) + kGemmWorkspaceBytes;
        unsigned char* w_bf = a_bf + bytes_a;
        // an A given as [K,M] is written as [M,K] while it is expanded: the tensor-core kernel streams a K-major A fastest
        int rc = a_is_km ? decode_transpose_bf16(Aq, a_bf, K, M, st) : hif8_decode(Aq, a_bf, HIF8_BF16, (size_t)M * K, 0, stream);
        if (rc == HIF8_OK) rc = hif8_decode(Wq, w_bf, HIF8_BF16, (size_t)K * N, 0, stream);
        if (rc != HIF8_OK) return rc;
        return launch_bf16_pair_gemm(a_bf, w_bf, w_is_nk, p, st);
    }
    // In between: room for A alone as BF16 (2 M K bytes; W, usually the larger operand, stays bytes).  A is expanded once
    // (as [M,K] whichever way it was given) and the fused kernel decodes only its W tiles; W may have any leading dimension.
    int a_mode = a_is_km ? 1 : 0;
    if (lda == (a_is_km ? M : K) && workspace_bytes >= kGemmWorkspaceBytes + bytes_a && !(reinterpret_cast<uintptr_t>(workspace) & 255)) {
        unsigned char* a_bf = reinterpret_cast<unsigned char*>(workspace) + kGemmWorkspaceBytes;
        const int rc = a_is_km ? decode_transpose_bf16(Aq, a_bf, K, M, st) : hif8_decode(Aq, a_bf, HIF8_BF16, (size_t)M * K, 0, stream);
        if (rc != HIF8_OK) return rc;
        // boxes of 64 k x 128 rows in the 128-byte-swizzled operand layout (a stack of one matrix: the pair form of the copy)
        if (!make_map3(&map_a, a_bf, (uint64_t)K, (uint64_t)M, 1, 0, BK, BM)) return HIF8_ERR_CUDA;
        a_mode = 2;
        if (w_is_nk) {
            // [N,K] weights: the swapped form, C^T = W^T A^T.  The weight rows are the operand that is decoded into tensor
            // memory, the expanded activations the one in shared memory; the kernel's M is N and its N is M.
            GemmParams q = p;
            q.M = N; q.N = M;
            q.c_by_tma = (c_dtype == HIF8_BF16 && !accumulate) ? 1 : 0;
            CUtensorMap map_cs;
            if (q.c_by_tma && !make_map(&map_cs, C, (uint64_t)N, (uint64_t)M, (uint64_t)ldc, 64, BM, true)) return HIF8_ERR_CUDA;
            q.tiles_m = (N + BM - 1) / BM; q.tiles_n = (M + BN - 1) / BN;
            const long long tiles2s = (long long)((N + 2 * BM - 1) / (2 * BM)) * q.tiles_n;
            if (tiles2s > 0x3FFFFFFF) return HIF8_ERR_SHAPE;
            CUtensorMap map_wb, map_ab;
            if (!make_map(&map_wb, Wq, (uint64_t)K, (uint64_t)N, (uint64_t)ldw, 2 * BK, BM, false, 128)) return HIF8_ERR_CUDA;  // rows of 128 k
            if (!make_map3(&map_ab, a_bf, (uint64_t)K, (uint64_t)M, 1, 0, BK, BN / 2)) return HIF8_ERR_CUDA;
            cudaLaunchConfig_t cs{};
            cs.gridDim = dim3(2u * (unsigned)tiles2s);
            cs.blockDim = dim3(kThreads);
            cs.dynamicSmemBytes = kSmemBytesSwapped;
            cs.stream = st;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            cs.attrs = at; cs.numAttrs = 1;
            const cudaError_t src = cudaLaunchKernelEx(&cs, hif8_gemm_kernel<0, true, true>, map_wb, map_ab, q.c_by_tma ? map_cs : map_ab, q);
            g_launches.fetch_add(1, std::memory_order_relaxed);
            return (src == cudaSuccess && cudaGetLastError() == cudaSuccess) ? HIF8_OK : HIF8_ERR_CUDA;
        }
    }

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2u * (unsigned)tiles2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = a_mode == 0 ? kSmemBytesWide : kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaError_t lrc;
    // BF16 results that replace C leave the [M,K]-activation kernel through tile stores (boxes of 64 columns x 128 rows)
    CUtensorMap map_c = map_a;  // (a valid map in any case; only read when c_by_tma is set)
    p.c_by_tma = (a_mode != 1 && c_dtype == HIF8_BF16 && !accumulate) ? 1 : 0;
    if (p.c_by_tma && !make_map(&map_c, C, (uint64_t)N, (uint64_t)M, (uint64_t)ldc, 64, BM, true)) return HIF8_ERR_CUDA;
    if (a_mode == 1) lrc = w_is_nk ? cudaLaunchKernelEx(&cfg, hif8_gemm_kernel<1, true>, map_a, map_w, map_c, p)
                                   : cudaLaunchKernelEx(&cfg, hif8_gemm_kernel<1, false>, map_a, map_w, map_c, p);
    else if (a_mode == 2) lrc = w_is_nk ? cudaLaunchKernelEx(&cfg, hif8_gemm_kernel<2, true>, map_a, map_w, map_c, p)
                                        : cudaLaunchKernelEx(&cfg, hif8_gemm_kernel<2, false>, map_a, map_w, map_c, p);
    else lrc = w_is_nk ? cudaLaunchKernelEx(&cfg, hif8_gemm_kernel<0, true>, map_a, map_w, map_c, p)
                       : cudaLaunchKernelEx(&cfg, hif8_gemm_kernel<0, false>, map_a, map_w, map_c, p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return (lrc == cudaSuccess && cudaGetLastError() == cudaSuccess) ? HIF8_OK : HIF8_ERR_CUDA;
}

extern "C" int hif8_gemm(const uint8_t* Aq, int64_t lda, const uint8_t* Wq, int64_t ldw, int w_is_nk, void* C, int64_t ldc,
                         int c_dtype, int M, int N, int K, const int* d_scale_exp_a, const int* d_scale_exp_w,
                         void* workspace, size_t workspace_bytes, hif8_stream_t stream)
{
    return gemm_entry(Aq, lda, 0, Wq, ldw, w_is_nk, C, ldc, c_dtype, M, N, K, d_scale_exp_a, d_scale_exp_w, nullptr, 0, workspace,
                      workspace_bytes, stream);
}

extern "C" int hif8_gemm_channel_scaled(const uint8_t* Aq, int64_t lda, const uint8_t* Wq, int64_t ldw, int w_is_nk, void* C,
                                        int64_t ldc, int c_dtype, int M, int N, int K, const int* d_scale_exp_a,
                                        const int* d_scale_exp_w_channel, void* workspace, size_t workspace_bytes,
                                        hif8_stream_t stream)
{
    if (!d_scale_exp_w_channel && M > 0 && N > 0) return HIF8_ERR_NULL;
    return gemm_entry(Aq, lda, 0, Wq, ldw, w_is_nk, C, ldc, c_dtype, M, N, K, d_scale_exp_a, nullptr, d_scale_exp_w_channel, 0,
                      workspace, workspace_bytes, stream);
}

extern "C" int hif8_gemm_ex(const uint8_t* Aq, int64_t lda, int a_is_km, const uint8_t* Wq, int64_t ldw, int w_is_nk, void* C,
                            int64_t ldc, int c_dtype, int M, int N, int K, const int* d_scale_exp_a, const int* d_scale_exp_w,
                            const int* d_scale_exp_w_channel, int accumulate, void* workspace, size_t workspace_bytes,
                            hif8_stream_t stream)
{
    return gemm_entry(Aq, lda, a_is_km ? 1 : 0, Wq, ldw, w_is_nk ? 1 : 0, C, ldc, c_dtype, M, N, K, d_scale_exp_a,
                      d_scale_exp_w_channel ? nullptr : d_scale_exp_w, d_scale_exp_w_channel, accumulate, workspace,
                      workspace_bytes, stream);
}

extern "C" int hif8_gemm_status(const void* workspace, hif8_stream_t stream)
{
    if (!workspace) return HIF8_ERR_NULL;
    int v = 0;
    if (cudaMemcpyAsync(&v, workspace, sizeof v, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess) return HIF8_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return HIF8_ERR_CUDA;
    return v == 0 ? HIF8_OK : HIF8_ERR_DEVICE_TIMEOUT;
}

extern "C" int hif8_last_device_status(hif8_stream_t stream)
{
    StatusKey k;
    std::memset(&k, 0, sizeof k);
    k.stream = (cudaStream_t)stream;
    StatusVal v;
    if (!g_last_status.find(k, &v)) return HIF8_OK;  // no GEMM-class call was made on this stream
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != v.dev) return HIF8_ERR_CUDA;
    return hif8_gemm_status(v.word, stream);
}

extern "C" int hif8_selftest_host_caches(int* failed_check)
{
    int check = 0;
    auto fail = [&](int c) { if (failed_check) *failed_check = c; return HIF8_ERR_SHAPE; };
    {   // set-up record: one initialisation per device ordinal, each with its own value
        static PerDevice<int> rec;
        static int calls;
        calls = 0;
        auto init = [](int dev, int* out) { calls++; *out = 1000 + dev; };
        const int* a = rec.get(3, init);
        const int* b = rec.get(5, init);
        const int* c = rec.get(3, init);
        check = 1; if (!a || !b || a != c || *a != 1003 || *b != 1005) return fail(check);
        check = 2; if (calls > 2) return fail(check);   // at most one per ordinal (zero when run before in this process)
        check = 3; if (rec.get(-1, init) || rec.get(kMaxDevices, init)) return fail(check);
    }
    {   // keyed cache: hit after miss, a failed build is not kept, the least recently used entry is replaced
        struct K { uint64_t a; uint32_t b; uint32_t pad; };
        LruCache<K, int, 4> cache;
        int builds = 0;
        auto make = [&](const K& k, int* v) { builds++; *v = (int)(k.a * 10 + k.b); return k.b != 99; };
        auto key = [](uint64_t a, uint32_t b) { K k; std::memset(&k, 0, sizeof k); k.a = a; k.b = b; return k; };
        int v = 0;
        check = 4; if (!cache.lookup_or_make(key(1, 2), &v, make) || v != 12 || builds != 1) return fail(check);
        check = 5; if (!cache.lookup_or_make(key(1, 2), &v, make) || v != 12 || builds != 1) return fail(check);
        check = 6; if (cache.lookup_or_make(key(7, 99), &v, make) || builds != 2) return fail(check);
        check = 7; if (cache.lookup_or_make(key(7, 99), &v, make) || builds != 3) return fail(check);
        for (uint64_t a = 2; a <= 4; a++) cache.lookup_or_make(key(a, 0), &v, make);   // cache now holds (1,2), 2, 3, 4
        check = 8; if (!cache.lookup_or_make(key(1, 2), &v, make) || builds != 6) return fail(check);   // refreshes (1,2)
        cache.lookup_or_make(key(5, 0), &v, make);                                     // replaces key 2, the oldest
        check = 9; if (builds != 7 || !cache.lookup_or_make(key(1, 2), &v, make) || builds != 7) return fail(check);
        check = 10; if (!cache.lookup_or_make(key(2, 0), &v, make) || builds != 8) return fail(check);
        check = 11; if (cache.hits() != 3 || cache.misses() != 6) return fail(check);
        int w = 0;
        cache.put(key(1, 2), 77);
        check = 12; if (!cache.find(key(1, 2), &w) || w != 77 || cache.find(key(42, 0), &w)) return fail(check);
    }
    if (failed_check) *failed_check = 0;
    return HIF8_OK;
}

extern "C" int hif8_selftest_wait_timeout(void* workspace, unsigned limit_ms, hif8_stream_t stream)
{
    if (!workspace) return HIF8_ERR_NULL;
    if (limit_ms == 0 || limit_ms > 1000) return HIF8_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(workspace, 0, 4, st) != cudaSuccess) return HIF8_ERR_CUDA;
    note_status_word(st, reinterpret_cast<const int*>(workspace));
    wait_selftest_kernel<<<1, 32, 0, st>>>(reinterpret_cast<int*>(workspace), (unsigned long long)limit_ms * 1000000ull);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? HIF8_OK : HIF8_ERR_CUDA;
}
