// Device-side helpers shared by the routing, scatter and combine kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace moe {

// Values of the device status word (mirrors moe_status where it applies).
constexpr int kDevOk = 0;
constexpr int kDevInsufficientExperts = 3;   // a token met fewer than k selectable experts
constexpr int kDevCapacity = 4;              // rows of an exchange did not fit the receive buffer
constexpr int kDevTimeout = 5;               // a bounded wait gave up

// Bounded waits: default number of polls before a waiter gives up (a context may carry
// another limit), and the back-off between polls of a flag in global memory.
// 1<<20 polls of >= 64 ns is well over 50 ms, far longer than any healthy step.
constexpr unsigned kDefaultSpinLimit = 1u << 20;
constexpr unsigned kSpinSleepNs = 64;

struct Control {
    unsigned ticket;     // next tile of the running routing kernel
    unsigned epoch;      // step counter tagging the per-tile count rows
    int status;          // kDev* code, sticky until the host clears it
    int pad;
};

// Programmatic dependent launch: let the next kernel of the stream be scheduled while this
// one is still running, and hold this kernel until the previous one has completed and its
// memory is visible.  Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void pdl_enter()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ unsigned lane_id() { return threadIdx.x & 31u; }

__device__ __forceinline__ unsigned lanemask_lt()
{
    unsigned m;
    asm volatile("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// A pair of 64-bit words moved by one 16-byte access at GPU scope.  Each word is read and
// written whole (a reader never sees half of one), which is all the look-back needs: every
// word carries its own validity tag.
__device__ __forceinline__ ulonglong2 ld_relaxed_v2_u64(const ulonglong2 *p)
{
    ulonglong2 v;
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_relaxed_v2_u64(ulonglong2 *p, unsigned long long a, unsigned long long b)
{
    asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(a), "l"(b) : "memory");
}

__device__ __forceinline__ int ld_relaxed_s32(const int *p)
{
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Hint: pull the cache line holding *p into L2.
__device__ __forceinline__ void prefetch_l2(const void *p)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// Asynchronous copies global -> shared that bypass registers; wait_all covers the calling
// thread's own copies (enough when the same thread reads what it asked for).
__device__ __forceinline__ void cp_async_16(void *smem_dst, const void *gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
                 : "memory");
}

__device__ __forceinline__ void cp_async_4(void *smem_dst, const void *gsrc)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
                 : "memory");
}

__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ void report_status(Control *ctl, int code)
{
    atomicCAS(&ctl->status, kDevOk, code);   // the first error wins and sticks
}

// 128-bit streaming accesses: the big rows are touched once per kernel, so they
// should not displace the small routing tables from L1.
__device__ __forceinline__ uint4 ld_stream_v4(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream_v4(uint4 *p, const uint4 &v)
{
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x),
                 "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// The same store with another cache policy, for measurements of what the write policy of the
// scatter does to the kernel that follows it: 1 = plain store, 2 = L2 evict-first hint,
// 3 = streaming (.cs) store.  0 is st_stream_v4.
__device__ __forceinline__ unsigned long long l2_policy_evict_first()
{
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

template <int POLICY>
__device__ __forceinline__ void st_policy_v4(uint4 *p, const uint4 &v, unsigned long long pol)
{
    if (POLICY == 1) {
        asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
    } else if (POLICY == 2) {
        asm volatile("st.global.L1::no_allocate.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(p), "r"(v.x),
                     "r"(v.y), "r"(v.z), "r"(v.w), "l"(pol)
                     : "memory");
    } else if (POLICY == 3) {
        asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
    } else {
        st_stream_v4(p, v);
    }
}

// ---------------------------------------------------------------------------
// exp / sigmoid from single IEEE fp32 operations (round to nearest even, never
// contracted, independent of compiler flags), so that sigmoid routing keys are
// reproducible bit for bit:
//   n = rint(z*log2e); r = z - n*ln2 (two fused steps); degree-7 Taylor
//   polynomial by Horner; scale by 2^n through the exponent field.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float exp_spec(float z)
{
    z = fminf(fmaxf(z, -87.0f), 88.0f);
    // rint by adding and removing 1.5 * 2^23: at that magnitude one ulp is 1, so the add rounds
    // z*log2e (|.| < 128) to the nearest integer, ties to even, and the subtraction is exact.
    // The integer itself sits in the low mantissa bits of the biased sum.
    const float biased = __fadd_rn(__fmul_rn(z, 0x1.715476p+0f), 12582912.0f);
    const float n = __fsub_rn(biased, 12582912.0f);
    float r = __fmaf_rn(-n, 0x1.62e430p-1f, z);
    r = __fmaf_rn(-n, -0x1.05c610p-29f, r);
    float p = 0x1.a01a02p-13f;
    p = __fmaf_rn(p, r, 0x1.6c16c2p-10f);
    p = __fmaf_rn(p, r, 0x1.111112p-7f);
    p = __fmaf_rn(p, r, 0x1.555556p-5f);
    p = __fmaf_rn(p, r, 0x1.555556p-3f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    const float two_n = __int_as_float((__float_as_int(biased) << 23) + 0x3f800000);   // (n + 127) << 23
    return __fmul_rn(p, two_n);
}

__device__ __forceinline__ float sigmoid_spec(float x)
{
    // 1 / d: the correctly rounded reciprocal is the correctly rounded quotient 1.0f / d
    return __frcp_rn(__fadd_rn(1.0f, exp_spec(-x)));
}

// Order-preserving map from fp32 to uint32 (larger float <=> larger integer),
// with -0 folded onto +0 (adding +0 in round-to-nearest turns -0 into +0 and
// changes nothing else) so that equal floats get equal codes.  0 is below the
// code of -inf and marks "already taken / not a candidate".
__device__ __forceinline__ uint32_t key_code(float f)
{
    const uint32_t u = __float_as_uint(__fadd_rn(f, 0.0f));
    return u ^ (static_cast<uint32_t>(static_cast<int32_t>(u) >> 31) | 0x80000000u);
}
constexpr uint32_t kCodeNegInf = 0x007FFFFFu;   // key_code(-inf)

// ---------------------------------------------------------------------------
// mbarrier and bulk asynchronous copies (the TMA engine moving whole row
// segments between global and shared memory without passing through registers)
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// global -> shared bulk copy, completion counted in bytes on an mbarrier
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, unsigned bytes,
                                          uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(smem_addr(smem_dst)),
        "l"(gsrc), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

// shared -> global bulk copy, tracked by the issuing thread's bulk async-group
__device__ __forceinline__ void bulk_store(void *gdst, const void *smem_src, unsigned bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_addr(smem_src)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

}  // namespace moe
