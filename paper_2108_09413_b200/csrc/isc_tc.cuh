// Inline-PTX wrappers for sm_100a shared by the tensor-core engines: mbarriers, bulk copies, tcgen05
// (tensor-memory allocation, MMA, commit, loads and stores), operand descriptors, the Philox4x32-10 block
// function and the inverse-CDF table search of the noise sampler (Def. 3.3, Eq. 2).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "isc_internal.h"

namespace isc {
namespace tc {

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// non-blocking test of a barrier phase
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// test that parks the thread in hardware for a bounded time when the phase is not complete
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void st_release(uint32_t addr, uint32_t v)
{
    asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint4 ld_acquire_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.acquire.cta.shared::cta.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void named_bar(int id, int n)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D = A * B (first K-step of a tile) and D += A * B
// True in exactly one lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred = 0;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\t@p mov.u32 %0, 1;\n\t}" : "+r"(pred));
    return pred != 0;
}
// A value every lane of the warp holds, in a form the compiler knows to be the same in all lanes.
__device__ __forceinline__ uint32_t warp_uniform(uint32_t v) { return __shfl_sync(0xffffffffu, v, 0); }

// The tensor-core instructions below are issued by one elected lane of a converged warp; their operands are
// computed by the whole warp from warp-uniform values.
__device__ __forceinline__ void mma_i8_first(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc)
{
    if (!elect_one()) return;
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc) : "memory");
}
__device__ __forceinline__ void mma_i8_acc(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc)
{
    if (!elect_one()) return;
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    if (!elect_one()) return;
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// asynchronous 16-column load of this thread's tensor-memory lane; the registers are valid after tmem_ld_wait()
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, int (&v)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int (&v)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// K-major, no-swizzle shared-memory operand descriptor: rows of 16 bytes, 8 rows contiguous,
// `sbo` bytes between 8-row groups, `lbo` bytes between the two 16-byte halves of K = 32.
__host__ __device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

// saturate four int32 to int8 and pack them (v0 in the low byte)
__device__ __forceinline__ uint32_t pack4_sat(int v0, int v1, int v2, int v3)
{
    uint32_t hi, d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(hi) : "r"(v3), "r"(v2));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(v1), "r"(v0), "r"(hi));
    return d;
}
// a * b + c as one 32x32+64 multiply-add
// Per-channel requantisation constants as stored in the blob: the 64-bit addend, then multiplier and shift.
// Loading the addend as one 64-bit register keeps it in an aligned register pair without any packing code.
struct ChanConst { long long B; int mult, s; };
__device__ __forceinline__ ChanConst ld_chan_const(uint32_t addr)
{
    long long b, ms;
    asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(b), "=l"(ms) : "r"(addr));
    ChanConst c;
    c.B = b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(c.mult), "=r"(c.s) : "l"(ms));
    return c;
}
__device__ __forceinline__ long long mad_wide(int a, int b, long long c)
{
    long long d;
    asm("mad.wide.s32 %0, %1, %2, %3;" : "=l"(d) : "r"(a), "r"(b), "l"(c));
    return d;
}
__device__ __forceinline__ int hi32(long long v)
{
    int lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
    return hi;
}
__device__ __forceinline__ int lo32(long long v)
{
    int lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
    return lo;
}
// byte K of w, sign-extended (one byte-permute with sign replication)
template <int K>
__device__ __forceinline__ int sbyte(uint32_t w)
{
    int d;
    asm("prmt.b32 %0, %1, 0, %2;" : "=r"(d) : "r"(w), "n"(((8 | K) << 12) | ((8 | K) << 8) | ((8 | K) << 4) | K));
    return d;
}

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c;
}

__device__ __forceinline__ int noise_level(uint32_t u, const uint32_t *__restrict__ cum, int T)
{
    int lo = 0, hi = 2 * T;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (u < __ldg(cum + mid)) hi = mid; else lo = mid + 1;
    }
    return lo - T;
}

// Inverse-CDF search min{ z : u < cum[z] } (the last entry always matches) by bisection between the guide table's
// results for the two uniforms that bracket u's top bits: the same result as the bisection over the whole table,
// in one or two steps for the bulk of the distribution.
__device__ __forceinline__ int noise_level_guided(uint32_t u, const uint32_t *__restrict__ cum, const uint32_t *__restrict__ guide, int T)
{
    const uint32_t j = u >> (32 - kNoiseGuideBits);
    uint32_t lo = __ldg(guide + j), hi = __ldg(guide + j + 1);
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if (u < __ldg(cum + mid)) hi = mid; else lo = mid + 1;
    }
    return (int)lo - T;
}

// The same search for the four uniforms of one Philox block with a fixed number of bisection steps (`steps` covers the
// widest guide interval; a step on an interval that has already closed changes nothing, since u < cum[result]), so
// that the four dependent load chains run interleaved.
__device__ __forceinline__ void noise_levels4(uint4 u4, const uint32_t *__restrict__ cum, const uint32_t *__restrict__ guide, int T,
                                              int steps, int (&z)[4])
{
    const uint32_t u[4] = {u4.x, u4.y, u4.z, u4.w};
    uint32_t lo[4], hi[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t j = u[k] >> (32 - kNoiseGuideBits);
        lo[k] = __ldg(guide + j);
        hi[k] = __ldg(guide + j + 1);
    }
    for (int s = 0; s < steps; ++s) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t mid = (lo[k] + hi[k]) >> 1;
            const bool below = u[k] < __ldg(cum + mid);
            hi[k] = below ? mid : hi[k];
            lo[k] = below ? lo[k] : min(mid + 1, hi[k]);
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) z[k] = (int)lo[k] - T;
}

// The same with both tables in shared memory (`cum_s`, `guide_s`: shared-memory addresses).  Thirty-two lanes searching
// a table in global memory touch up to thirty-two cache lines per load; in shared memory the same load costs its bank
// conflicts only.
__device__ __forceinline__ void noise_levels4_shared(uint4 u4, uint32_t cum_s, uint32_t guide_s, int T, int steps, int (&z)[4])
{
    const uint32_t u[4] = {u4.x, u4.y, u4.z, u4.w};
    uint32_t lo[4], hi[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t j = u[k] >> (32 - kNoiseGuideBits);
        lo[k] = lds32(guide_s + 4u * j);
        hi[k] = lds32(guide_s + 4u * j + 4u);
    }
    for (int s = 0; s < steps; ++s) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t mid = (lo[k] + hi[k]) >> 1;
            const bool below = u[k] < lds32(cum_s + 4u * mid);
            hi[k] = below ? mid : hi[k];
            lo[k] = below ? lo[k] : min(mid + 1, hi[k]);
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) z[k] = (int)lo[k] - T;
}

}  // namespace tc
}  // namespace isc
