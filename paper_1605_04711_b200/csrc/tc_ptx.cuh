// Inline-PTX building blocks shared by the tensor-core kernels: mbarriers with bounded waits,
// TMA tensor copies, tcgen05 (MMA issue, commit, fences, tensor-memory load/store) and the
// shared-memory operand descriptors.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "twn.h"

namespace {

constexpr unsigned long long kWaitLimitNs = 1000000000ull;
constexpr int kConvergedTries = 16;   // warp-wide blocking probes before a single lane takes over

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(void *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(void *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(2000u) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test(void *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false when the limit ran out or another role gave up.
// Waiting warps share their scheduler with the warps that do the work, so a waiter backs
// off with nanosleep instead of polling flat out (`backoff_ns` = 0 for the latency-critical
// waits of the MMA warp, which rely on the suspend time of try_wait alone).
__device__ __forceinline__ bool mbar_wait(void *bar, uint32_t parity, volatile int *abort_flag, int32_t *status,
                                          uint32_t backoff_ns = 64, unsigned long long limit_ns = kWaitLimitNs)
{
    if (mbar_try(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if (backoff_ns) __nanosleep(backoff_ns);
        if ((spin & 255u) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) {
                *abort_flag = 1;
                if (status) atomicMin(status, (int)TWN_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// Warp-wide wait: lane 0 polls, the result is broadcast.  One polling lane instead of 32
// keeps the shared-memory pipe free for the warps that are working.
__device__ __forceinline__ bool mbar_wait_warp(void *bar, uint32_t parity, volatile int *abort_flag, int32_t *status,
                                               uint32_t backoff_ns = 64, unsigned long long limit_ns = kWaitLimitNs)
{
    // fast path: the phase is already over.  One non-blocking probe by the whole warp and one vote:
    // measured at 16 cycles, against 46 for the potentially blocking try_wait and 129 when a single
    // lane probes and the result is shuffled (the divergent region costs more than the 31 probes).
    if (__all_sync(0xffffffffu, mbar_test(bar, parity))) return true;
    // not yet: one potentially blocking probe by the whole warp (the hardware suspends the warp for a
    // while if the phase is about to end), before the single-lane loop below
#pragma unroll 1
    for (int i = 0; i < kConvergedTries; ++i)
        if (__all_sync(0xffffffffu, mbar_try(bar, parity))) return true;
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status, backoff_ns, limit_ns) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    __syncwarp();
    return ok != 0;
}

__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, void *bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, const void *src, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }


// The MMA warp runs its loops converged; tcgen05.mma and tcgen05.commit are issued by the
// lane that elect.sync picks, with the predicate applied inside the asm block (measured to be
// the cheapest way to issue: no divergent region around the instruction).
// D[tmem] (+)= A[tmem] * B[smem]^T, bf16 x bf16 -> fp32.
template <bool ACC>
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p, pe;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "n"(ACC ? 1 : 0)
        : "memory");
}

__device__ __forceinline__ void tc_commit(void *bar)
{
    asm volatile(
        "{\n\t.reg .pred pe;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(smem_u32(bar)) : "memory");
}

// One k-block: four K=16 MMAs.  FIRST clears the accumulator with the first of them.  The
// accumulate flag is a compile-time constant so that no predicate has to be built at run time:
// whatever the issuing thread executes between two MMAs is time the tensor core may sit idle.
template <bool FIRST>
__device__ __forceinline__ void tc_mma_block(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc)
{
    tc_mma_ts<!FIRST>(d_tmem, a_tmem, b_desc, idesc);
    tc_mma_ts<true>(d_tmem, a_tmem + 8, b_desc + 2, idesc);
    tc_mma_ts<true>(d_tmem, a_tmem + 16, b_desc + 4, idesc);
    tc_mma_ts<true>(d_tmem, a_tmem + 24, b_desc + 6, idesc);
}

// Read-only global loads that the compiler neither moves nor wraps in control flow.
__device__ __forceinline__ void ld_nc_v4(uint4 &v, const uint32_t *p)
{
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
}
__device__ __forceinline__ void ld_nc_v2(uint32_t &x, uint32_t &y, const uint32_t *p)
{
    asm volatile("ld.global.nc.v2.u32 {%0, %1}, [%2];" : "=r"(x), "=r"(y) : "l"(p));
}
__device__ __forceinline__ void ld_nc_u32(uint32_t &v, const uint32_t *p)
{
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(p));
}

// K-major, 128-byte swizzled operand tile: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);   // start address
    d |= (uint64_t)1 << 16;                     // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset
    d |= (uint64_t)1 << 46;                     // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                     // 128-byte swizzle
    return d;
}

// kind::f16 instruction descriptor: bf16 A and B (both K-major), fp32 accumulate.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N)
{
    return (1u << 4)              // D format fp32
           | (1u << 7)            // A format bf16
           | (1u << 10)           // B format bf16
           | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// Waits for the tensor-memory loads of this thread.  The registers of the load that is being
// waited for are passed through the statement, so that the compiler keeps every use of them
// behind the wait even when another load was issued in between.
__device__ __forceinline__ void tmem_wait_ld(uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization attribute may start once
// every block of the kernel before it in the stream has called pdl_launch_dependents() (or exited); what it does
// before pdl_wait() must not touch global memory that the earlier kernel writes or reads, and pdl_wait() returns
// when the earlier kernel has completed and its writes are visible.  Without the attribute both are no-ops.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Two fp32 values -> one bf16x2 word (round to nearest even), `lo` in the low half.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t pk;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(hi), "f"(lo));
    return pk;
}
// Same, negative values clamped to zero (a NaN stays a NaN).
__device__ __forceinline__ uint32_t pack_bf16x2_relu(float lo, float hi)
{
    uint32_t pk;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(hi), "f"(lo));
    return pk;
}
// (x0, x1) <- (x0 * a0 + b0, x1 * a1 + b1), both lanes in one instruction.
__device__ __forceinline__ void fma_f32x2(uint32_t &x0, uint32_t &x1, float a0, float a1, float b0, float b1)
{
    unsigned long long x, a, b;
    asm("mov.b64 %0, {%1, %2};" : "=l"(x) : "r"(x0), "r"(x1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "f"(b0), "f"(b1));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(x) : "l"(x), "l"(a), "l"(b));
    asm("mov.b64 {%0, %1}, %2;" : "=r"(x0), "=r"(x1) : "l"(x));
}

// Element pair j (0..7) of a packed code word -> two bf16 values in {-2, 0, +2}.  The pair's
// fields sit 2*j bits below the top of the two half-words (bit 0 of a field = non-zero, bit 1 =
// sign); shifted to the top they are the sign and the high exponent bit of a bf16, and
// 0x4000 is 2.0.  The factor 2 is taken out again with the scale of the epilogue, so a decoded
// pair costs one shift and one mask.  (Field 10 would read as -0.)
constexpr float kDecodedUnit = 2.0f;
__device__ __forceinline__ uint32_t pair_to_bf16x2(uint32_t w, int j)
{
    return (w << (2 * j)) & 0xC000C000u;
}

// Binary codes, one bit per weight (1 = -1): element pair j (0..15) of a word has its two bits j below the
// top of the two half-words; shifted to the top they are the sign bits of a bf16 pair, and 0x3F80 is 1.0.
// One shift and one three-input logic operation per pair; the decoded values are exactly +-1.
__device__ __forceinline__ uint32_t pair_to_bf16x2_b1(uint32_t w, int j)
{
    return ((w << j) & 0x80008000u) | 0x3F803F80u;
}
// The 64 codes of one k-block -> 32 bf16 pairs.  BITS = 2: four words of ternary codes (values +-2 / 0);
// BITS = 1: two words of binary codes (values +-1).
template <int BITS>
__device__ __forceinline__ void decode_kblock(const uint32_t (&wv)[4], uint32_t (&out)[32])
{
    if (BITS == 2) {
#pragma unroll
        for (int g = 0; g < 4; ++g)
#pragma unroll
            for (int e = 0; e < 8; ++e) out[g * 8 + e] = pair_to_bf16x2(wv[g], e);
    } else {
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
            for (int e = 0; e < 16; ++e) out[g * 16 + e] = pair_to_bf16x2_b1(wv[g], e);
    }
}
// what a decoded +1 is worth: taken out again with the scale of the epilogue
template <int BITS> __host__ __device__ constexpr float decoded_unit() { return BITS == 2 ? kDecodedUnit : 1.0f; }

// ---------------------------------------------------------------- the kernel

// D[tmem] (+)= A[smem] * B[smem]^T, both operands through shared-memory descriptors.
template <bool ACC>
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p, pe;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "n"(ACC ? 1 : 0)
        : "memory");
}

// MN-major, 128-byte swizzled operand: the MN index runs along 128-byte rows (64 bf16), eight
// K rows form a 1024-byte group, `mn_block_bytes` separates consecutive 64-element MN blocks.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t saddr, uint32_t mn_block_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((mn_block_bytes >> 4) & 0x3FFFu) << 16;   // leading byte offset: next MN block
    d |= (uint64_t)(1024 >> 4) << 32;                         // stride byte offset: next 8 K rows
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Same, with the distance between consecutive 8-row K groups given as well.  A tile with a halo
// serves several taps at once: the groups are 8-pixel runs of image rows (`k_group_bytes` = one
// halo row when a tile row is 8 pixels wide) and the "next MN block" is the same tile one pixel
// further (128 bytes).  The swizzle is a function of the absolute shared-memory address, so the
// start may be any 128-byte row of a 1024-byte aligned buffer.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128_groups(uint32_t saddr, uint32_t mn_block_bytes, uint32_t k_group_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((mn_block_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((k_group_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// kind::f16 instruction descriptor, bf16 operands both MN-major, fp32 accumulate.
__host__ __device__ constexpr uint32_t make_idesc_mn(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

}  // namespace
