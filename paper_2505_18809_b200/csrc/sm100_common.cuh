// Device helpers shared by the tcgen05 attention kernels (sm_100a): mbarrier and tensor-memory
// primitives as inline PTX, bounded waits, the shared-memory matrix descriptor, and the arithmetic
// of one 64-column stretch of a softmax row.
#pragma once

#include <cuda/ptx>

#include "vorta_internal.h"

namespace vorta {
namespace sm100 {

namespace ptx = cuda::ptx;

constexpr float kRescaleThreshold = 8.0f;  // log2 units a row maximum may exceed the reference before O is rescaled
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(bar),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait on a phase of an mbarrier.  Returns false if the CTA is aborting.  Ctl is the kernel's
// control block in shared memory: `volatile int32_t abort`, and `kStatusBase`, which tells the kernels'
// codes apart in the status word.
template <class Ctl>
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, Ctl *ctl, int32_t *status, int32_t code)
{
    const unsigned long long t0 = global_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0) {
            if (ctl->abort) return false;
            if (global_ns() - t0 > kWaitLimitNs) {
                ctl->abort = code;
                atomicCAS(status, 0, Ctl::kStatusBase + code);
                return false;
            }
        }
    }
}

template <class Ctl>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, Ctl *ctl, int32_t *status, int32_t code)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, status, code);
}

// The same wait with a warp-uniform result, and a warp-uniform copy of a value all
// lanes hold: both come out of warp-wide reductions, which the compiler can keep in
// uniform registers.  The MMA warp needs this: the operands of tcgen05.mma are uniform
// registers, and only provably uniform values and control flow reach them without a
// per-instruction detour through vector registers.
template <class Ctl>
__device__ __forceinline__ bool mbar_wait_uniform(uint32_t bar, uint32_t parity, Ctl *ctl, int32_t *status,
                                                  int32_t code)
{
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, ctl, status, code)) != 0;
}

__device__ __forceinline__ uint32_t uniform_u32(uint32_t v) { return __reduce_max_sync(0xffffffffu, v); }

__device__ __forceinline__ uint32_t elect_one()
{
    uint32_t leader;
    asm volatile(
        "{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(leader));
    return leader;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }


// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
// lbo/sbo in bytes: for a K-major operand sbo is the pitch of 8-row groups; for an
// MN-major operand lbo is the pitch of 64-element column blocks and sbo the pitch
// of 8-row (K) groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;  // version
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// acc.x += low bf16 of w, acc.y += high bf16 of w: the mixed-precision add takes the bf16 operand as it
// is (exact in fp32), so the packed word needs no shift and mask to be summed
__device__ __forceinline__ void add_bf16x2(float2 &acc, uint32_t w)
{
    unsigned short lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(w));
    asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(acc.x) : "h"(lo));
    asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(acc.y) : "h"(hi));
}

// exp2(s * scale - ref) for 64 scores of a row, packed two bf16 per word IN
// PLACE into s[0 .. 32): a packed word never lands on a score still to be read.
// The row sums take the ROUNDED values the PV MMA will use, so that O / sum stays a true
// weighted mean of V rows (with the unrounded ones a row that attends to a single key is
// off by up to 2^-9 of |v|, beyond the output tolerance).  Scale-and-shift uses the packed
// two-wide fp32 fma; the sums take the bf16 halves of the packed words directly (mixed-precision
// add: one instruction per score, against a shift, a mask and half a packed add before; measured
// 2.4 % of a layer at 118 800 tokens).
template <bool kAll = true>
__device__ __forceinline__ void exp_block(uint32_t (&s)[64], float scale, float neg_ref, float2 (&sum)[2], int32_t width = 64)
{
    const float2 sc = make_float2(scale, scale), nr = make_float2(neg_ref, neg_ref);
#pragma unroll
    for (int c = 0; c < 64; c += 4) {
        if (!kAll && c >= width) break;  // a narrow sub-block: the columns past its width are not needed (width: a multiple of 16)
        float2 x0 = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc, nr);
        float2 x1 = __ffma2_rn(make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sc, nr);
        const uint32_t k0 = pack_bf16(ex2(x0.x), ex2(x0.y));
        const uint32_t k1 = pack_bf16(ex2(x1.x), ex2(x1.y));
        s[c >> 1] = k0;
        s[(c >> 1) + 1] = k1;
        add_bf16x2(sum[0], k0);
        add_bf16x2(sum[1], k1);
    }
}

// this thread's row of O times a
template <int D>
__device__ __forceinline__ void rescale_o(uint32_t t_o, float a)
{
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        ptx::tcgen05_ld_32x32b(o, t_o + c * 32);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * a);
        ptx::tcgen05_st_32x32b(t_o + c * 32, o);
    }
}

// maximum of the 64 scores of a sub-block (four independent chains of three-input max)
__device__ __forceinline__ float row_max64(const uint32_t (&s)[64])
{
    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
    for (int c = 0; c < 64; c += 8) {
        mx0 = max3(mx0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
        mx1 = max3(mx1, __uint_as_float(s[c + 2]), __uint_as_float(s[c + 3]));
        mx2 = max3(mx2, __uint_as_float(s[c + 4]), __uint_as_float(s[c + 5]));
        mx3 = max3(mx3, __uint_as_float(s[c + 6]), __uint_as_float(s[c + 7]));
    }
    return fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
}

}  // namespace sm100
}  // namespace vorta
