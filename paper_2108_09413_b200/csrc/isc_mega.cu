// Shared-memory-resident tensor-core engine (sm_100a) for CIFAR-shaped residual networks.
//
// One persistent CTA per SM carries a group of G noisy samples through the whole network:
// the activations never leave shared memory, every 3x3 / 1x1 convolution is an implicit GEMM
// on tcgen05 (kind::i8, int32 accumulators in tensor memory), and only vote counts return to
// global memory.  Per group the CTA runs a list of phases prepared on the host:
//
//   FILL   set a freshly allocated activation region to its halo value (the zero-point)
//   INPUT  draw the discrete Gaussian noise (Def. 3.3, Eq. 2), add it to the image, saturate to
//          0..255 and write the result straight into the first layer's operand region (Def. 3.4)
//   CONV   tiles of 128 positions x N output channels: one thread issues the MMAs of a tile,
//          four epilogue warps requantise it (fixed-point multiplier, shift, zero-points,
//          residual add, clamp) and write the next layer's operand
//   TAIL   global average pool, FC, argmax and vote per sample (Algorithm 1 steps 1-4)
//
// Activation layout: [channel plane of 16][position][16 bytes]; a position is a pixel of the
// zero-point-padded image, all samples of the group stacked in one linear index with one halo
// row/column shared between neighbours, so a filter tap is a constant byte offset and eight
// consecutive positions are one 8x16-byte core matrix of the no-swizzle K-major operand layout.
//
// Every device-side wait is bounded by a wall-clock limit; on expiry the CTA raises an abort
// flag, all remaining waits fall through, and the host reports ISC_ERR_TIMEOUT.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <vector>

#include "isc_mega.h"

namespace isc {

namespace {

#ifdef ISC_TRACE
// Timeline instrumentation, compiled only with -DISC_TRACE: CTA 0 records (warp and event, round, SM clock)
// for the rounds in [g_trace_lo, g_trace_hi).
constexpr unsigned kTraceMax = 16384;
__device__ unsigned long long g_trace[3 * kTraceMax];
__device__ unsigned int g_trace_n, g_trace_lo, g_trace_hi;
__device__ __forceinline__ void trace(int ev, uint32_t r)
{
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && r >= g_trace_lo && r < g_trace_hi) {
        const unsigned i = atomicAdd(&g_trace_n, 1u);
        if (i < kTraceMax) {
            g_trace[3 * i] = (unsigned long long)(ev | ((threadIdx.x >> 5) << 8));
            g_trace[3 * i + 1] = r;
            g_trace[3 * i + 2] = (unsigned long long)clock64();
        }
    }
}
#else
#define trace(ev, r) ((void)0)
#endif

constexpr int kIssuers = 4;                 // warps 0..3: an elected lane of each issues the MMAs of every 4th tile
constexpr int kEpiWarps = 8;                // warps 4..11: epilogue, two warpgroups of "fat" threads (168 registers)
constexpr int kWarpGroups = kEpiWarps / 4;
constexpr int kThreads = 32 * (kIssuers + kEpiWarps);
// Tensor memory is used as two halves of 256 columns.  A CONV phase is cut into rounds of consecutive tiles
// (as many as fit a half: 16, 8 or 4 tiles of 16, 32 or 64 columns); rounds take the halves in turn over the
// whole run of the kernel.  The four issuing warps share the tiles of a round; the eight epilogue warps share
// its outputs.  FILL, INPUT and TAIL phases are rounds of their own without tensor-core work, so that one
// sequence number orders everything that happens to a group.
constexpr int kHalves = 2, kHalfCols = 256;
constexpr int kMaxFusedCols = 64;
// accumulator columns of a tile with n output channels
__host__ __device__ constexpr int tile_columns(int n) { return n <= 16 ? 16 : n <= 32 ? 32 : 64; }
static_assert(kWarpGroups == 2, "the epilogue splits a round's work between two warpgroups");
constexpr int kMaxKsteps = 20;
constexpr int kMaxChunks = 4;
constexpr int kMaxPhases = 136;
constexpr int kCtrlBytes = 4096;
constexpr int kSmemLimit = 227 * 1024;
constexpr int kFillItemBytes = 8192;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait

enum { PH_FILL = 0, PH_INPUT = 1, PH_CONV = 2, PH_TAIL = 3 };
enum { ERR_NONE = 0, ERR_WAIT_ITEMS = 1, ERR_WAIT_WEIGHTS = 2, ERR_WAIT_EMPTY = 3, ERR_WAIT_FULL = 4,
       ERR_WAIT_DRAIN = 5 };

// Where and how one group of 16 output channels of a CONV phase is written.
struct alignas(16) ChunkInfo {
    uint32_t out_off, res_off;      // byte offsets of the destination / residual channel plane
    int32_t lo;                     // lower clamp when flags bit 0 is set
    uint32_t halo;                  // zero-point byte replicated: value of positions outside the image
    uint32_t flags, pad0, pad1, pad2;   // bit0 explicit lower clamp, bit1 residual add
};

// Host-side description of a phase (the planner's working form).
struct alignas(16) MPhase {
    int32_t kind, n_items, item_base, full_sync;
    int32_t H, W, Wp, HsWp;                 // geometry of the positions this phase walks (CONV: its input tensor)
    int32_t P_first, scatter, o_Wp, o_HsWp;
    uint32_t magic_hswp, magic_wp, pad0, pad1;
    uint32_t fill_off, fill_bytes, fill_word, pad2;
    uint32_t in_off, n_ksteps, idesc, n_chunks;
    uint32_t w_off, w_bytes, const_off, conv_index;
    int32_t n_tiles, n_rows;
    int32_t res_mult, res_n;
    int32_t n_rounds, tiles_per_round;      // CONV: how the tiles are cut into rounds
    long long res_R;
    int32_t a_delta[kMaxKsteps];
    uint32_t a_lbo[kMaxKsteps];
    ChunkInfo chunk[kMaxChunks];
};

// ---- what the kernel reads -------------------------------------------------------------------

// One entry per phase, copied to shared memory when the kernel starts.
//   CONV: n_items = rounds | tiles per round << 8 | accumulator columns per tile << 16, a = shared-memory offset of
//         the phase's blob (ConvDesc, weights, per-channel constants), b = tiles
//   FILL: a = offset of the region, b = bytes | halo byte << 24
struct alignas(16) PhaseEntry { uint32_t kind_sync, n_items, a, b; };     // kind | full_sync << 8 | chunks << 16

// Where the blob of convolution c comes from (global) and goes to (shared).
struct alignas(16) ConvSrc { unsigned long long gmem; uint32_t bytes_phase, smem_off; };   // bytes | phase << 24

// Head of every blob: everything the issuing threads and the epilogue need to know about the phase.
struct alignas(16) ConvDesc {
    uint32_t in_off, n_ksteps, idesc, n_rows;
    int32_t P_first, HsWp, Wp, scatter;
    int32_t o_Wp, o_HsWp;
    uint32_t magic_hswp, magic_wp;
    uint32_t n_chunks, weights_rel, consts_rel, mode;   // mode: epilogue variant, same for all chunks
    int32_t res_mult, res_n;
    long long res_R;
    ChunkInfo chunk[kMaxChunks];
    int32_t a_delta[kMaxKsteps];
    uint32_t a_lbo[kMaxKsteps];
    uint32_t pad1[4];
};
static_assert(sizeof(ConvDesc) % 128 == 0, "blob sections must stay 128-byte aligned");

struct FcConst { int32_t mult, n, zp_out, lo, bias, pad0, pad1, pad2; };

struct MegaParams {
    const PhaseEntry *ptab;
    const ConvSrc *conv_src;
    int32_t n_phases, n_conv, rounds_per_group, pad_r;
    int32_t in_H, in_W, in_Wp, in_HsWp;
    int32_t G, n_groups, n_samples, in_c;
    const uint8_t *x;                 // clean image, CHW
    NoiseStream ns;
    uint32_t input_off;               // operand region of the first layer
    int32_t input_halo;
    // tail
    uint32_t tail_in_off, tail_plane_bytes;
    int32_t tail_C, tail_H, tail_W, tail_Wp, tail_HsWp;
    int32_t pool_mult, pool_n, pool_zp_in, pool_zp_out, pool_lo;
    const int8_t *fc_w;               // [n_classes][64]
    const FcConst *fc_c;
    int32_t n_classes, fc_pad;
    int32_t *counts;
    int8_t *logits;                   // [n_samples][n_classes] or null
    int32_t *err;
    // debug
    int32_t stop_phase;
    uint32_t dump_off, dump_bytes;
    uint8_t *dump;
};

struct Ctrl {
    unsigned long long full[kHalves], done[kHalves], wbar[3], drain;
    uint32_t tmem_base;
    volatile int abort_flag;
    int32_t hist[128];
    PhaseEntry ptab[kMaxPhases];
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// ------------------------------------------------------------------ PTX wrappers

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

// ------------------------------------------------------------------ bounded waits

struct Waiter {
    Ctrl *ctrl;
    int32_t *err;
    __device__ __forceinline__ bool aborted() const { return ctrl->abort_flag != 0; }
    __device__ __noinline__ void fail(int code)
    {
        ctrl->abort_flag = 1;
        atomicCAS(err, 0, code | (blockIdx.x << 8));
    }
    // Wait for a phase of an mbarrier.  Each attempt parks the thread in hardware for a bounded time,
    // so a waiting warp does not compete for issue slots.
    __device__ __forceinline__ bool barrier(uint32_t bar, uint32_t parity, int code)
    {
        if (mbar_test(bar, parity)) return true;
        const unsigned long long t0 = globaltimer();
        for (int spin = 0;; ++spin) {
            if (mbar_try(bar, parity)) return true;
            if ((spin & 7) == 7) {
                if (aborted()) return false;
                if (globaltimer() - t0 > kWaitLimitNs) { fail(code); return false; }
            }
        }
    }
    // Wait on a predicate over shared-memory progress counters, backing off between polls.
    template <typename Pred>
    __device__ __forceinline__ bool until(Pred pred, int code)
    {
        if (pred()) return true;
        const unsigned long long t0 = globaltimer();
        for (int spin = 0;; ++spin) {
            __nanosleep(64);
            if (pred()) return true;
            if ((spin & 31) == 31) {
                if (aborted()) return false;
                if (globaltimer() - t0 > kWaitLimitNs) { fail(code); return false; }
            }
        }
    }
};

// Every epilogue warp publishes the index of the next item it has work in: all counters >= need means items
// 0..need-1 are complete.  One 16-byte acquire read per warpgroup.
// ------------------------------------------------------------------ rounds
//
// Everything that happens to a group is a sequence of rounds, numbered over the whole run of the kernel:
// a CONV phase contributes n_rounds of them (consecutive tiles), every other phase one.  Round r uses
// tensor-memory half r & 1 and the barrier pair full[r & 1] / done[r & 1]; each of the two completes exactly
// once per round (also for rounds without tensor-core work), so the parity to wait for is (r >> 1) & 1.
//   full[h]: the four issuing warps have committed their tiles of the round (or simply arrived)
//   done[h]: the eight epilogue warps have stored the round's outputs (and no longer read the half)
// A role only ever waits for the latest or the one-before-latest completion of a barrier, so a parity is
// never ambiguous.  Rounds complete in order.  Round r may start when round r - 2 is complete (its half is
// free) and its operands are there: `dep`, the latest round whose outputs it reads, is r - 1 at most.

// dependency of round k (tiles [k tpr, (k+1) tpr)) of a CONV phase whose first round is `first`:
//   with full_sync, everything before the phase; else the producing phase (the one just before, cut into rounds
//   the same way) up to its round k + 1, because a tile reads one tile beyond itself
__device__ __forceinline__ uint32_t round_dep(uint32_t first, int k, int n_rounds, bool full_sync)
{
    return full_sync ? first - 1u : first - (uint32_t)n_rounds + (uint32_t)min(k + 1, n_rounds - 1);
}

// ------------------------------------------------------------------ issuing warps

__device__ __forceinline__ void issue_weights(const ConvSrc *src, uint32_t sbase, uint32_t wbar_addr)
{
    const uint4 v = __ldg(reinterpret_cast<const uint4 *>(src));
    const void *gmem = reinterpret_cast<const void *>(((unsigned long long)v.y << 32) | v.x);
    const uint32_t bytes = v.z & 0xFFFFFFu;
    mbar_expect_tx(wbar_addr, bytes);
    bulk_g2s(sbase + v.w, gmem, bytes, wbar_addr);
}

struct IssueArgs {
    uint32_t desc, a0, w0, n_rows, idesc, first, tile_cols;
    int n_rounds, tpr, n_tiles, issuer, full_sync;
};

// wait until round r may be issued: its half is free (round r - 2 complete) and round `dep` is complete
__device__ __forceinline__ bool round_start_wait(Waiter w, Ctrl *ctrl, uint32_t r, uint32_t dep)
{
    const uint32_t h = r & 1u;
    if (r >= 2u && !w.barrier(smem_u32(&ctrl->done[h]), ((r - 2u) >> 1) & 1u, ERR_WAIT_EMPTY)) return false;
    if (r >= 1u && dep == r - 1u && !w.barrier(smem_u32(&ctrl->done[h ^ 1u]), ((r - 1u) >> 1) & 1u, ERR_WAIT_ITEMS)) return false;
    return true;
}

// The rounds of one CONV phase with KS K-steps per tile.  The issuing warp takes every fourth tile of a round.
// The low words of the operand descriptors stay in registers; tile t is 128 t positions, i.e. 128 t units of the
// A descriptors' start-address field, further.
template <int KS>
__device__ __forceinline__ bool issue_phase(Waiter w, Ctrl *ctrl, uint32_t tmem, const IssueArgs &ia)
{
    uint32_t alo[KS], blo[KS];
    const uint32_t ahi = (uint32_t)(make_desc(0, 0, 128) >> 32), bhi = (uint32_t)(make_desc(0, 128, 256) >> 32);
#pragma unroll
    for (int k = 0; k < KS; ++k) {
        const uint32_t delta = warp_uniform(lds32(ia.desc + offsetof(ConvDesc, a_delta) + 4 * k));
        const uint32_t lbo = warp_uniform(lds32(ia.desc + offsetof(ConvDesc, a_lbo) + 4 * k));
        alo[k] = (uint32_t)make_desc(ia.a0 + delta, lbo, 128);
        blo[k] = (uint32_t)make_desc(ia.w0 + (uint32_t)k * ia.n_rows * 32u, 128, 256);
    }
    const uint32_t idesc = ia.idesc, tile_cols = ia.tile_cols;
    const int n_tiles = ia.n_tiles, tpr = ia.tpr, issuer = ia.issuer;
    for (int k = 0; k < ia.n_rounds; ++k) {
        const uint32_t r = ia.first + (uint32_t)k, h = r & 1u;
        if (!round_start_wait(w, ctrl, r, round_dep(ia.first, k, ia.n_rounds, ia.full_sync))) return false;
        trace(1, r);
        tc_fence_after();
        const int t0 = k * tpr, t1 = min(n_tiles, t0 + tpr);
        const uint32_t d0 = tmem + h * kHalfCols;
#pragma unroll 1
        for (int t = t0 + issuer; t < t1; t += kIssuers) {
            const uint32_t d = d0 + (uint32_t)(t - t0) * tile_cols;
#pragma unroll
            for (int q = 0; q < KS; ++q) {
                const uint64_t ad = ((uint64_t)ahi << 32) | (uint64_t)(alo[q] + 128u * (uint32_t)t);
                const uint64_t bd = ((uint64_t)bhi << 32) | (uint64_t)blo[q];
                if (q == 0) mma_i8_first(d, ad, bd, idesc);
                else mma_i8_acc(d, ad, bd, idesc);
            }
        }
        mma_commit(smem_u32(&ctrl->full[h]));        // arrives at once when this warp had no tile in the round
        trace(2, r);
    }
    return true;
}

// Same for an arbitrary number of K-steps (descriptors rebuilt from shared memory for every tile).
__device__ __noinline__ bool issue_phase_any(Waiter w, Ctrl *ctrl, uint32_t tmem, const IssueArgs &ia, uint32_t n_ksteps)
{
    for (int k = 0; k < ia.n_rounds; ++k) {
        const uint32_t r = ia.first + (uint32_t)k, h = r & 1u;
        if (!round_start_wait(w, ctrl, r, round_dep(ia.first, k, ia.n_rounds, ia.full_sync))) return false;
        tc_fence_after();
        const int t0 = k * ia.tpr, t1 = min(ia.n_tiles, t0 + ia.tpr);
        for (int t = t0 + ia.issuer; t < t1; t += kIssuers) {
            const uint32_t d = tmem + h * kHalfCols + (uint32_t)(t - t0) * ia.tile_cols;
            for (uint32_t q = 0; q < n_ksteps; ++q) {
                const uint32_t delta = warp_uniform(lds32(ia.desc + offsetof(ConvDesc, a_delta) + 4 * q));
                const uint32_t lbo = warp_uniform(lds32(ia.desc + offsetof(ConvDesc, a_lbo) + 4 * q));
                const uint64_t ad = make_desc(ia.a0 + delta + 2048u * (uint32_t)t, lbo, 128);
                const uint64_t bd = make_desc(ia.w0 + q * ia.n_rows * 32u, 128, 256);
                if (q == 0) mma_i8_first(d, ad, bd, ia.idesc);
                else mma_i8_acc(d, ad, bd, ia.idesc);
            }
        }
        mma_commit(smem_u32(&ctrl->full[h]));
    }
    return true;
}

// Warps 0..3, all lanes converged: the tensor-core work of one group
__device__ __noinline__ void mma_role(const MegaParams &p, Ctrl *ctrl, uint32_t sbase, uint32_t tmem, int it, int issuer)
{
    Waiter w{ctrl, p.err};
    const uint32_t ptab = smem_u32(ctrl->ptab);
    const uint32_t conv_off = (uint32_t)it * p.n_conv;
    const int n_phases = p.n_phases, stop_phase = p.stop_phase, n_conv = p.n_conv;
    const ConvSrc *conv_src = p.conv_src;
    const bool leader = issuer == 0 && elect_one();         // the one thread that starts the weight copies
    uint32_t r_next = (uint32_t)it * p.rounds_per_group;      // sequence number of the next round
    uint32_t conv_index = 0;
    bool first_round = true;
    for (int ph = 0; ph < n_phases && ph <= stop_phase; ++ph) {
        uint4 e = ld_shared_v4(ptab + 16 * ph);
        e.x = warp_uniform(e.x); e.y = warp_uniform(e.y); e.z = warp_uniform(e.z); e.w = warp_uniform(e.w);
        const int kind = e.x & 0xFF, full_sync = (e.x >> 8) & 1;
        if (kind != PH_CONV) {
            // a round without tensor-core work: keep the barriers in step
            const uint32_t r = r_next++;
            if (!round_start_wait(w, ctrl, r, r - 1u)) return;
            if (first_round) {
                // everything of the previous group is complete: the ring slot of this group's first weights is free
                if (leader && !w.aborted()) issue_weights(conv_src, sbase, smem_u32(&ctrl->wbar[conv_off % 3]));
                __syncwarp();
                first_round = false;
            }
            if (elect_one()) mbar_arrive(smem_u32(&ctrl->full[r & 1u]));
            __syncwarp();
            continue;
        }
        const int n_rounds = (int)(e.y & 0xFF), tpr = (int)((e.y >> 8) & 0xFF);
        const uint32_t cg = conv_off + conv_index;
        // operands and the ring slot of the next weights: wait for the first round's start conditions here, so
        // that the copy of the next phase's weights is under way before this phase's tiles are issued
        if (!round_start_wait(w, ctrl, r_next, round_dep(r_next, 0, n_rounds, full_sync))) return;
        if (leader && (int)conv_index + 1 < n_conv) {
            const ConvSrc *nxt = conv_src + conv_index + 1;
            if ((int)(__ldg(&nxt->bytes_phase) >> 24) <= stop_phase)
                issue_weights(nxt, sbase, smem_u32(&ctrl->wbar[(cg + 1) % 3]));
        }
        __syncwarp();
        if (!w.barrier(smem_u32(&ctrl->wbar[cg % 3]), (cg / 3) & 1, ERR_WAIT_WEIGHTS)) return;
        // phase parameters from the head of the blob
        const uint32_t desc = sbase + e.z;
        uint4 h = ld_shared_v4(desc);                              // in_off, n_ksteps, idesc, n_rows
        h.x = warp_uniform(h.x); h.y = warp_uniform(h.y); h.z = warp_uniform(h.z); h.w = warp_uniform(h.w);
        IssueArgs ia;
        ia.desc = desc;
        ia.a0 = sbase + h.x + warp_uniform(lds32(desc + offsetof(ConvDesc, P_first))) * 16u;
        ia.w0 = desc + warp_uniform(lds32(desc + offsetof(ConvDesc, weights_rel)));
        ia.n_rows = h.w; ia.idesc = h.z; ia.n_rounds = n_rounds; ia.tpr = tpr; ia.n_tiles = (int)e.w;
        ia.tile_cols = (e.y >> 16) & 0xFF;
        ia.first = r_next; ia.full_sync = full_sync; ia.issuer = issuer;
        bool ok;
        switch (h.y) {
        case 1: ok = issue_phase<1>(w, ctrl, tmem, ia); break;
        case 5: ok = issue_phase<5>(w, ctrl, tmem, ia); break;
        case 9: ok = issue_phase<9>(w, ctrl, tmem, ia); break;
        case 18: ok = issue_phase<18>(w, ctrl, tmem, ia); break;
        default: ok = issue_phase_any(w, ctrl, tmem, ia, h.y); break;
        }
        if (!ok) return;
        conv_index += 1;
        r_next += (uint32_t)n_rounds;
        first_round = false;
    }
}

// ------------------------------------------------------------------ epilogue warps

struct EpiCtx {
    Ctrl *ctrl;
    uint32_t sbase, tmem;
    int warp_e, wg, quarter, lane, tid_wg;
};

__device__ void fill_item(uint32_t fill_off, uint32_t bytes_halo, const EpiCtx &c, int i)
{
    const uint32_t fill_bytes = bytes_halo & 0xFFFFFFu, word = (bytes_halo >> 24) * 0x01010101u;
    const uint32_t begin = (uint32_t)i * kFillItemBytes;
    const uint32_t end = min(begin + kFillItemBytes, fill_bytes);
    const uint4 v = make_uint4(word, word, word, word);
    for (uint32_t o = begin + c.tid_wg * 16; o < end; o += 128 * 16) st_shared_v4(c.sbase + fill_off + o, v);
}

// INPUT: one thread = four horizontally adjacent pixels of one sample, all input channels.
__device__ void input_item(const MegaParams &p, const EpiCtx &c, int i, int grp)
{
    const int H = p.in_H, W = p.in_W, Wp = p.in_Wp, HsWp = p.in_HsWp, G = p.G, in_c = p.in_c;
    const int wq = W >> 2;
    const int quads = G * H * wq;
    const int qi = i * 128 + c.tid_wg;
    if (qi >= quads) return;
    const int s = qi / (H * wq);
    const int rem = qi - s * (H * wq);
    const int y = rem / wq, x4 = rem - y * wq;
    const long long j = p.ns.first_sample + (long long)grp * G + s;
    const uint32_t *__restrict__ cum = p.ns.cum;
    const int T = p.ns.T;
    const uint32_t key0 = p.ns.key0, key1 = p.ns.key1, ctr2 = p.ns.ctr2;
    const uint32_t ctr3 = p.ns.ctr3_fixed | (uint32_t)(((j >> 32) & 0xFF) << 8);
    const uint8_t *__restrict__ x = p.x;
    uint32_t px[4] = {0, 0, 0, 0};
    for (int ch = 0; ch < in_c; ++ch) {
        const uint32_t e = (uint32_t)((ch * H + y) * W + 4 * x4);
        const uint4 r = philox4x32_10(make_uint4(e >> 2, (uint32_t)(j & 0xFFFFFFFFll), ctr2, ctr3), key0, key1);
        const uint32_t u[4] = {r.x, r.y, r.z, r.w};
        const uint32_t clean = __ldg(reinterpret_cast<const uint32_t *>(x + e));
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            int v = (int)((clean >> (8 * k)) & 0xFF) + noise_level(u[k], cum, T);
            v = min(255, max(0, v));
            px[k] |= (uint32_t)v << (8 * ch);
        }
    }
    const uint32_t pos = (uint32_t)(s * HsWp + (y + 1) * Wp + 4 * x4 + 1);
    const uint32_t dst = c.sbase + p.input_off;
#pragma unroll
    for (int k = 0; k < 4; ++k) st_shared_v4(dst + (pos + k) * 16u, make_uint4(px[k], 0, 0, 0));
}

// What the epilogue warps keep in registers for the whole of a CONV phase.
struct ConvRegs {
    int P_first, HsWp, Wp, scatter, o_Wp, o_HsWp, G;
    uint32_t magic_hswp, magic_wp, const_addr, n_chunks, chunks;
    int res_mult, res_sh;          // res_sh = n - 32 when n >= 32, else n
    long long res_R;
    uint32_t mode;                 // bit0 explicit lower clamp, bit1 residual, bit2 residual shift >= 32
};

// desc = shared-memory address of the phase's ConvDesc
__device__ __forceinline__ ConvRegs load_conv_regs(uint32_t desc, int G)
{
    ConvRegs r;
    const uint4 g0 = ld_shared_v4(desc + offsetof(ConvDesc, P_first));      // P_first, HsWp, Wp, scatter
    const uint4 g1 = ld_shared_v4(desc + offsetof(ConvDesc, o_Wp));         // o_Wp, o_HsWp, magic_hswp, magic_wp
    const uint4 g2 = ld_shared_v4(desc + offsetof(ConvDesc, n_chunks));     // n_chunks, weights_rel, consts_rel, mode
    const uint4 g3 = ld_shared_v4(desc + offsetof(ConvDesc, res_mult));     // res_mult, res_n, res_R
    r.P_first = (int)g0.x; r.HsWp = (int)g0.y; r.Wp = (int)g0.z; r.scatter = (int)g0.w;
    r.o_Wp = (int)g1.x; r.o_HsWp = (int)g1.y; r.magic_hswp = g1.z; r.magic_wp = g1.w;
    r.n_chunks = g2.x; r.const_addr = desc + g2.z; r.mode = g2.w;
    r.res_mult = (int)g3.x; r.res_sh = (int)g3.y >= 32 ? (int)g3.y - 32 : (int)g3.y;
    r.res_R = (long long)(((unsigned long long)g3.w << 32) | g3.z);
    r.G = G;
    r.chunks = desc + offsetof(ConvDesc, chunk);
    return r;
}

// One output channel:
//   main    : y = floor((acc * mult + B) / 2^(32 + s)); B holds the folded bias, the rounding half and the
//             output zero-point, so this is rs(acc' * mult, 31 + shift) + zp_out exactly
//   residual: y += floor((r * res_mult + R) / 2^n), R = 2^(n-1) - zp_res * res_mult   (kResHigh: n >= 32)
template <bool kRes, bool kResHigh, bool kLo, int K>
__device__ __forceinline__ int requant1(int acc, const ChanConst &cs, uint32_t rword, const ConvRegs &R, int lo)
{
    int y = hi32(mad_wide(acc, cs.mult, cs.B)) >> cs.s;
    if (kRes) {
        const long long t = mad_wide(sbyte<K>(rword), R.res_mult, R.res_R);
        y += kResHigh ? (hi32(t) >> R.res_sh) : (int)__funnelshift_r((uint32_t)lo32(t), (uint32_t)hi32(t), R.res_sh);
    }
    if (kLo) y = max(y, lo);
    return y;
}

// Where the positions of this thread (one per tile of the super-tile) are, and where their results go.
template <int SUP>
struct Spots {
    uint32_t pos[SUP], opos[SUP];
    uint32_t keep, store;            // bit j: tile j keeps its computed value (else halo) / is stored at all
};

template <int SUP>
__device__ __forceinline__ Spots<SUP> locate(const ConvRegs &R, const EpiCtx &c, int st, int n_tiles)
{
    Spots<SUP> sp;
    sp.keep = 0; sp.store = 0;
#pragma unroll
    for (int j = 0; j < SUP; ++j) {
        const int t = st * SUP + j;
        // a tile beyond the phase's last one is never stored; it borrows the last tile's addresses so that
        // every read stays inside the tensor's region
        const uint32_t pos = (uint32_t)(R.P_first + 128 * min(t, n_tiles - 1) + c.quarter * 32 + c.lane);
        // position -> (sample, row, column) of the padded image
        const uint32_t s = __umulhi(pos, R.magic_hswp);
        const uint32_t rem = pos - s * (uint32_t)R.HsWp;
        const uint32_t y1 = __umulhi(rem, R.magic_wp);
        const uint32_t x1 = rem - y1 * (uint32_t)R.Wp;
        const bool interior = (int)s < R.G && y1 >= 1 && x1 >= 1;
        bool store = t < n_tiles;
        uint32_t opos = pos;
        if (R.scatter) {
            const uint32_t y = y1 - 1, x = x1 - 1;
            store = store && interior && !(y & 1) && !(x & 1);
            opos = s * (uint32_t)R.o_HsWp + ((y >> 1) + 1) * (uint32_t)R.o_Wp + (x >> 1) + 1;
        }
        sp.pos[j] = pos; sp.opos[j] = opos;
        if (R.scatter || interior) sp.keep |= 1u << j;
        if (store) sp.store |= 1u << j;
    }
    return sp;
}

// Requantise one 16-channel chunk of the tiles of a super-tile (16 SUP accumulators per thread) and store it.
// The per-channel constants are read once and applied to all SUP positions.
template <bool kRes, bool kResHigh, bool kLo, int SUP>
__device__ __forceinline__ void chunk_compute(const int (&acc)[SUP][16], const ConvRegs &R, const EpiCtx &c,
                                              const Spots<SUP> &sp, uint32_t ch)
{
    const uint4 ci = ld_shared_v4(R.chunks + ch * (uint32_t)sizeof(ChunkInfo));   // out_off, res_off, lo, halo
    const uint32_t cbase = R.const_addr + ch * 256u;
    const int lo = (int)ci.z;
    uint32_t rw[SUP][4];
#pragma unroll
    for (int j = 0; j < SUP; ++j) {
        uint4 rv = make_uint4(0, 0, 0, 0);
        if (kRes) rv = ld_shared_v4(c.sbase + ci.y + sp.pos[j] * 16u);
        rw[j][0] = rv.x; rw[j][1] = rv.y; rw[j][2] = rv.z; rw[j][3] = rv.w;
    }
    uint32_t out[SUP][4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const ChanConst c0 = ld_chan_const(cbase + (4 * g + 0) * 16), c1 = ld_chan_const(cbase + (4 * g + 1) * 16);
        const ChanConst c2 = ld_chan_const(cbase + (4 * g + 2) * 16), c3 = ld_chan_const(cbase + (4 * g + 3) * 16);
#pragma unroll
        for (int j = 0; j < SUP; ++j) {
            const int y0 = requant1<kRes, kResHigh, kLo, 0>(acc[j][4 * g + 0], c0, rw[j][g], R, lo);
            const int y1 = requant1<kRes, kResHigh, kLo, 1>(acc[j][4 * g + 1], c1, rw[j][g], R, lo);
            const int y2 = requant1<kRes, kResHigh, kLo, 2>(acc[j][4 * g + 2], c2, rw[j][g], R, lo);
            const int y3 = requant1<kRes, kResHigh, kLo, 3>(acc[j][4 * g + 3], c3, rw[j][g], R, lo);
            out[j][g] = pack4_sat(y0, y1, y2, y3);
        }
    }
#pragma unroll
    for (int j = 0; j < SUP; ++j) {
        uint4 o = make_uint4(out[j][0], out[j][1], out[j][2], out[j][3]);
        if (!((sp.keep >> j) & 1u)) o = make_uint4(ci.w, ci.w, ci.w, ci.w);
        if ((sp.store >> j) & 1u) st_shared_v4(c.sbase + ci.x + sp.opos[j] * 16u, o);
    }
}

// End of a round for an epilogue warp: its shared-memory writes become visible to the tensor cores' reads, its
// tensor-memory reads are ordered before the arrival, and the round counts as complete once all eight warps are here.
__device__ __forceinline__ void round_done(const EpiCtx &c, uint32_t r)
{
    tc_fence_before();
    fence_proxy_async();
    __syncwarp();
    if (c.lane == 0) mbar_arrive(smem_u32(&c.ctrl->done[r & 1u]));
    trace(4, r);
}

// The rounds of one CONV phase.  A warp owns 32 rows (its tensor-memory lanes) of every tile; the two warpgroups
// split a round's tiles pair by pair when the phase has one 16-channel chunk, and chunk by chunk otherwise, so
// that both have the same amount of work in every round.  The loops over pairs and chunks are kept rolled on
// purpose: their body (32 outputs per thread) is a few KB of code and stays in the instruction cache; a fully
// unrolled round does not and leaves the warps waiting for instruction fetches.
template <bool kRes, bool kResHigh, bool kLo>
__device__ __noinline__ void conv_phase_rounds(Waiter w, const EpiCtx &c_in, const ConvRegs &R_in, int n_rounds, int tpr,
                                               int n_tiles, uint32_t first, uint32_t tile_cols)
{
    // private copies: values reached through references would be re-read after every barrier or fence
    const EpiCtx c = c_in;
    const ConvRegs R = R_in;
    const uint32_t lane_base = c.tmem + ((uint32_t)(c.quarter * 32) << 16);
    const uint32_t n_chunks = R.n_chunks;
    const bool by_chunk = (n_chunks & 1u) == 0;
    const uint32_t ch0 = by_chunk ? (uint32_t)c.wg : 0u, ch_step = by_chunk ? (uint32_t)kWarpGroups : 1u;
    bool ok = true;
    for (int k = 0; k < n_rounds; ++k) {
        const uint32_t r = first + (uint32_t)k, h = r & 1u;
        const int t0 = k * tpr, t1 = min(n_tiles, t0 + tpr);
        if (ok) ok = w.barrier(smem_u32(&c.ctrl->full[h]), (r >> 1) & 1u, ERR_WAIT_FULL);
        ok = __all_sync(0xffffffffu, ok);
        trace(3, r);
        tc_fence_after();
        const uint32_t half_addr = lane_base + h * kHalfCols;
        const int n_pairs = (t1 - t0 + 1) >> 1;
#pragma unroll 1
        for (int pr = by_chunk ? 0 : c.wg; pr < n_pairs; pr += by_chunk ? 1 : kWarpGroups) {
            // t0 is even, so pair pr of the round is pair t0 / 2 + pr of the phase; tiles from t1 on are not stored
            const Spots<2> sp = locate<2>(R, c, (t0 >> 1) + pr, t1);
            const uint32_t pair_addr = half_addr + (uint32_t)(2 * pr) * tile_cols;
#pragma unroll 1
            for (uint32_t ch = ch0; ch < n_chunks; ch += ch_step) {
                int acc[2][16];
                tmem_ld16_issue(pair_addr + ch * 16, acc[0]);
                tmem_ld16_issue(pair_addr + tile_cols + ch * 16, acc[1]);
                tmem_ld_wait();
                if (ok) chunk_compute<kRes, kResHigh, kLo, 2>(acc, R, c, sp, ch);
            }
        }
        round_done(c, r);
    }
}

__device__ __forceinline__ void conv_phase_dispatch(Waiter w, const EpiCtx &c, const ConvRegs &R, int n_rounds, int tpr,
                                                    int n_tiles, uint32_t first, uint32_t tile_cols)
{
    switch (R.mode & 7u) {
    case 0: conv_phase_rounds<false, false, false>(w, c, R, n_rounds, tpr, n_tiles, first, tile_cols); break;
    case 1: conv_phase_rounds<false, false, true>(w, c, R, n_rounds, tpr, n_tiles, first, tile_cols); break;
    case 2: conv_phase_rounds<true, false, false>(w, c, R, n_rounds, tpr, n_tiles, first, tile_cols); break;
    case 3: conv_phase_rounds<true, false, true>(w, c, R, n_rounds, tpr, n_tiles, first, tile_cols); break;
    case 6: conv_phase_rounds<true, true, false>(w, c, R, n_rounds, tpr, n_tiles, first, tile_cols); break;
    default: conv_phase_rounds<true, true, true>(w, c, R, n_rounds, tpr, n_tiles, first, tile_cols); break;
    }
}

// TAIL: global average pool, FC, argmax and vote; one warp carries one sample.
__device__ void tail_sample(const MegaParams &p, const EpiCtx &c, int s, bool counted_slot, int grp)
{
    const int tail_H = p.tail_H, tail_W = p.tail_W, tail_C = p.tail_C, tail_Wp = p.tail_Wp, tail_HsWp = p.tail_HsWp;
    const int n_classes = p.n_classes;
    const int hw = tail_H * tail_W;
    int pooled[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int ch = c.lane + 32 * h;
        int q = 0;
        if (ch < tail_C) {
            const uint32_t base = c.sbase + p.tail_in_off + (uint32_t)(ch >> 4) * p.tail_plane_bytes + (ch & 15);
            int sum = 0;
            for (int i = 0; i < hw; ++i) {
                const int y = i / tail_W, x = i - y * tail_W;
                const uint32_t pos = (uint32_t)(s * tail_HsWp + (y + 1) * tail_Wp + x + 1);
                int v;
                asm volatile("ld.shared.s8 %0, [%1];" : "=r"(v) : "r"(base + pos * 16u));
                sum += v - p.pool_zp_in;
            }
            long long v = ((long long)sum * p.pool_mult + (1ll << (p.pool_n - 1))) >> p.pool_n;
            v += p.pool_zp_out;
            v = v < p.pool_lo ? p.pool_lo : v;
            v = v > 127 ? 127 : v;
            q = (int)v;
        }
        pooled[h] = q;
    }
    const long long sample = (long long)grp * p.G + s;          // index within this launch
    const bool counted = counted_slot && sample < p.n_samples;
    int best_v = -1000, best_o = 0x7fffffff;
    for (int o0 = 0; o0 < n_classes; o0 += 32) {
        const int o = o0 + c.lane;
        const bool live = o < n_classes;
        const FcConst k = p.fc_c[live ? o : 0];
        const int8_t *wrow = p.fc_w + (size_t)(live ? o : 0) * 64;
        int acc = k.bias;
        for (int cc = 0; cc < tail_C; ++cc) {
            const int a = __shfl_sync(0xffffffffu, pooled[cc >> 5], cc & 31);
            acc += a * (int)__ldg(wrow + cc);
        }
        long long v = ((long long)acc * k.mult + (1ll << (k.n - 1))) >> k.n;
        v += k.zp_out;
        v = v < k.lo ? k.lo : v;
        v = v > 127 ? 127 : v;
        if (live) {
            if ((int)v > best_v) { best_v = (int)v; best_o = o; }
            if (counted && p.logits) p.logits[sample * n_classes + o] = (int8_t)v;
        }
    }
    // lowest index among the maxima
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        const int ov = __shfl_xor_sync(0xffffffffu, best_v, d), oo = __shfl_xor_sync(0xffffffffu, best_o, d);
        if (ov > best_v || (ov == best_v && oo < best_o)) { best_v = ov; best_o = oo; }
    }
    if (counted && c.lane == 0) atomicAdd(&c.ctrl->hist[best_o], 1);
}

// Epilogue warps: all non-tensor-core work of one group.  Item g of a FILL / INPUT / TAIL phase belongs to
// warpgroup g mod 2; the outputs of a CONV round are split as described above.
__device__ __noinline__ void epi_role(const MegaParams &p, EpiCtx &c, int it, int grp)
{
    Waiter w{c.ctrl, p.err};
    const uint32_t ptab = smem_u32(c.ctrl->ptab);
    const uint32_t conv_off = (uint32_t)it * p.n_conv;
    const int n_phases = p.n_phases, stop_phase = p.stop_phase, G = p.G;
    uint32_t r_next = (uint32_t)it * p.rounds_per_group, conv_index = 0;
    for (int ph = 0; ph < n_phases && ph <= stop_phase; ++ph) {
        const uint4 e = ld_shared_v4(ptab + 16 * ph);
        const int kind = e.x & 0xFF;
        bool ok;
        if (kind == PH_CONV) {
            const int n_rounds = (int)(e.y & 0xFF), tpr = (int)((e.y >> 8) & 0xFF);
            const uint32_t cg = conv_off + conv_index, first = r_next;
            conv_index += 1;
            r_next += (uint32_t)n_rounds;
            ok = w.barrier(smem_u32(&c.ctrl->wbar[cg % 3]), (cg / 3) & 1, ERR_WAIT_WEIGHTS);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {                       // keep the barriers in step so that nobody waits for this warp
                for (int k = 0; k < n_rounds; ++k) round_done(c, first + (uint32_t)k);
                continue;
            }
            const ConvRegs R = load_conv_regs(c.sbase + e.z, G);
            conv_phase_dispatch(w, c, R, n_rounds, tpr, (int)e.w, first, (e.y >> 16) & 0xFF);
            continue;
        }
        // a round of its own: every earlier round must be complete in all warps, then the items are shared out
        const uint32_t r = r_next++;
        const int n_items = (int)e.y;
        ok = r == 0u || w.barrier(smem_u32(&c.ctrl->done[(r & 1u) ^ 1u]), ((r - 1u) >> 1) & 1u, ERR_WAIT_ITEMS);
        ok = __all_sync(0xffffffffu, ok);
        trace(5 + kind, r);
        for (int i = c.wg; i < n_items; i += kWarpGroups) {
            if (!ok) break;
            if (kind == PH_FILL) {
                fill_item(e.z, e.w, c, i);
            } else if (kind == PH_INPUT) {
                input_item(p, c, i, grp);
            } else {
                const int s = i * 4 + (c.warp_e & 3);
                tail_sample(p, c, min(s, G - 1), s < G, grp);
            }
        }
        round_done(c, r);
    }
}

__global__ void __launch_bounds__(kThreads, 1) k_mega(const __grid_constant__ MegaParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem);
    const uint32_t sbase = smem_u32(smem);
    const int warp = (int)warp_uniform(threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kHalves; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), kIssuers);      // every issuing warp commits (or arrives) once per round
            mbar_init(smem_u32(&ctrl->done[s]), kEpiWarps);     // every epilogue warp arrives once per round
        }
        for (int s = 0; s < 3; ++s) mbar_init(smem_u32(&ctrl->wbar[s]), 1);
        mbar_init(smem_u32(&ctrl->drain), kIssuers);
        ctrl->abort_flag = 0;
    }
    for (int i = threadIdx.x; i < 128; i += blockDim.x) ctrl->hist[i] = 0;
    for (int i = threadIdx.x; i < p.n_phases; i += blockDim.x) ctrl->ptab[i] = p.ptab[i];
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), 512);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctrl->tmem_base;

    EpiCtx c;
    c.ctrl = ctrl; c.sbase = sbase; c.tmem = tmem;
    c.warp_e = warp - kIssuers; c.wg = (warp - kIssuers) >> 2; c.quarter = warp & 3; c.lane = lane;
    c.tid_wg = ((warp - kIssuers) & 3) * 32 + lane;

    int it = 0;
    for (int grp = blockIdx.x; grp < p.n_groups; grp += gridDim.x, ++it) {
        if (warp < kIssuers) {
            mma_role(p, ctrl, sbase, tmem, it, warp);
        } else {
            epi_role(p, c, it, grp);
        }
        __syncthreads();
    }
    if (!ctrl->abort_flag)
        for (int i = threadIdx.x; i < p.n_classes; i += blockDim.x)
            if (ctrl->hist[i]) atomicAdd(p.counts + i, ctrl->hist[i]);
    if (p.dump)
        for (uint32_t o = threadIdx.x * 16u; o < p.dump_bytes; o += blockDim.x * 16u)
            *reinterpret_cast<uint4 *>(p.dump + o) = ld_shared_v4(sbase + p.dump_off + o);
    // no tensor-core work may be in flight when tensor memory is released
    if (warp < kIssuers) {
        Waiter w{ctrl, p.err};
        __syncwarp();
        mma_commit(smem_u32(&ctrl->drain));          // by the lane that issued this warp's tensor-core work
        w.barrier(smem_u32(&ctrl->drain), 0, ERR_WAIT_DRAIN);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// =============================================================================== host planner

struct PlanTensor {
    int C = 0, H = 0, W = 0, planes = 0, halo = 0;
    int Wp = 0, HsWp = 0, P_first = 0, n_tiles = 0, npa = 0;
    uint32_t plane_bytes = 0, bytes = 0;
    int buffer = -1;             // index into buffers
    int producer_phase = -1;
    bool scatter_produced = false;
    int last_use_layer = -1;     // model layer index of the last reader
};

struct PlanBuffer {
    uint32_t bytes = 0, off = 0;
    int birth = 0, death = 0;    // phase indices
    int halo = 0;
    int C = 0, H = 0, W = 0;
    int last_tenant_death_layer = -1;
    bool last_death_as_conv_operand = false;
};

struct AllocReq { uint32_t bytes; int birth, death, slack; uint32_t *off; };

void set_geometry(PlanTensor &t, int G)
{
    t.planes = (t.C + 15) / 16;
    t.Wp = t.W + 1;
    t.HsWp = (t.H + 1) * t.Wp;
    t.P_first = t.Wp + 1;
    const int p_last = (G - 1) * t.HsWp + t.H * t.Wp + t.W;
    t.n_tiles = (p_last - t.P_first + 1 + 127) / 128;
    t.npa = (t.P_first + 128 * t.n_tiles + t.Wp + 2 + 7) & ~7;
    t.plane_bytes = (uint32_t)t.npa * 16u;
    t.bytes = t.plane_bytes * (uint32_t)t.planes;
}

uint32_t magic_for(uint32_t d, uint32_t limit, bool *ok)
{
    const uint32_t m = (uint32_t)(((1ull << 32) + d - 1) / d);
    for (uint32_t p = 0; p < limit; ++p)
        if ((uint32_t)(((unsigned long long)p * m) >> 32) != p / d) { *ok = false; break; }
    return m;
}

}  // namespace

struct MegaPlan {
    int G = 0, in_c = 0, in_h = 0, in_w = 0, n_classes = 0;
    std::vector<MPhase> phases;
    std::vector<int> conv_phase;
    int rounds_per_group = 0;
    uint32_t smem_bytes = 0;
    MegaParams base;                      // fields that do not change between launches
    // device copies
    PhaseEntry *d_ptab = nullptr;
    ConvSrc *d_conv_src = nullptr;
    uint8_t *d_blob = nullptr;
    int8_t *d_fc_w = nullptr;
    FcConst *d_fc_c = nullptr;
    int32_t *d_err = nullptr;
    uint8_t *d_dump = nullptr;
    // model tensor id -> where it lives (for the debug read-back)
    std::vector<PlanTensor> tensors;
    std::vector<uint32_t> tensor_off;
    int sm_count = 0;
    bool attr_set = false;
};

namespace {

struct ConvNode {
    int layer;                 // model layer index
    int fused_layer = -1;      // second layer (1x1 projection) sharing input and stride
};

bool conv_ok(const isc_layer &L, bool first)
{
    if (L.op != ISC_CONV2D) return false;
    if (L.kh != L.kw || (L.kh != 1 && L.kh != 3)) return false;
    if (L.pad != (L.kh - 1) / 2) return false;
    if (L.stride != 1 && L.stride != 2) return false;
    if (first) { if (L.cin > 4 || L.stride != 1) return false; }
    else if (L.cin % 16 != 0 || L.cin > 64) return false;
    if (L.cout % 16 != 0 || L.cout > 64) return false;
    return true;
}

// First-fit placement of one request among the allocations that are still busy at its birth.
bool place(std::vector<AllocReq> &done, AllocReq &r, uint32_t capacity)
{
    std::vector<std::pair<uint32_t, uint32_t>> busy;
    for (const AllocReq &e : done)
        if (e.death >= r.birth - r.slack) busy.push_back({*e.off, *e.off + e.bytes});
    std::sort(busy.begin(), busy.end());
    uint32_t at = kCtrlBytes;
    for (const auto &b : busy) {
        if (at + r.bytes <= b.first) break;
        at = std::max(at, (b.second + 127u) & ~127u);
    }
    if (at + r.bytes > capacity) return false;
    *r.off = at;
    done.push_back(r);
    return true;
}

// Build the phase list for groups of G samples.  Returns false when it does not fit.
bool plan_for_G(const MegaLayerIn *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes, int G,
                MegaPlan *plan, std::vector<uint8_t> *blob_out, std::vector<uint32_t> *blob_offsets)
{
    const int n_conv_layers = n_layers - 2;
    // ---- tensors of the model (tensor t = output of layer t-1)
    std::vector<PlanTensor> T((size_t)n_layers + 1);
    T[0].C = in_c; T[0].H = in_h; T[0].W = in_w; T[0].halo = layers[0].d.zp_in;
    for (int i = 0; i < n_conv_layers; ++i) {
        const isc_layer &L = layers[i].d;
        const PlanTensor &in = T[(size_t)L.in_tensor];
        PlanTensor &o = T[(size_t)i + 1];
        o.C = L.cout;
        o.H = (in.H + 2 * L.pad - L.kh) / L.stride + 1;
        o.W = (in.W + 2 * L.pad - L.kw) / L.stride + 1;
        o.halo = L.zp_out;
        if (L.stride == 2 && ((in.H & 1) || (in.W & 1))) return false;
    }
    for (int t = 0; t <= n_conv_layers; ++t) set_geometry(T[(size_t)t], G);
    for (int i = 0; i < n_layers; ++i) {
        T[(size_t)layers[i].d.in_tensor].last_use_layer = i;
        if (layers[i].d.res_tensor >= 0) T[(size_t)layers[i].d.res_tensor].last_use_layer = i;
    }
    // ---- conv nodes, fusing a 3x3 with the 1x1 projection that follows it on the same input
    std::vector<ConvNode> nodes;
    for (int i = 0; i < n_conv_layers; ++i) {
        ConvNode nd; nd.layer = i;
        if (i + 1 < n_conv_layers) {
            const isc_layer &A = layers[i].d, &B = layers[i + 1].d;
            if (A.kh == 3 && B.kh == 1 && B.in_tensor == A.in_tensor && B.stride == A.stride && B.res_tensor < 0 &&
                A.res_tensor < 0 && A.cout + B.cout <= kMaxFusedCols && A.zp_in == B.zp_in &&
                T[(size_t)i + 1].H == T[(size_t)i + 2].H && T[(size_t)i + 1].W == T[(size_t)i + 2].W) {
                nd.fused_layer = i + 1;
                ++i;
            }
        }
        nodes.push_back(nd);
    }
    // ---- phase skeleton: FILL(input) INPUT, then per node [FILL per fresh output] CONV, then TAIL
    struct Skel { int kind; int node; int tensor; };
    std::vector<Skel> skel;
    std::vector<PlanBuffer> buffers;
    std::vector<int> layer_phase((size_t)n_layers, -1);
    auto new_buffer = [&](int tensor) {
        PlanBuffer b;
        b.bytes = T[(size_t)tensor].bytes; b.halo = T[(size_t)tensor].halo;
        b.C = T[(size_t)tensor].C; b.H = T[(size_t)tensor].H; b.W = T[(size_t)tensor].W;
        b.birth = (int)skel.size();
        buffers.push_back(b);
        T[(size_t)tensor].buffer = (int)buffers.size() - 1;
        skel.push_back({PH_FILL, -1, tensor});
    };
    new_buffer(0);
    skel.push_back({PH_INPUT, -1, 0});
    int prev_conv_layer_last = -1;         // last model layer covered by the previous conv phase
    for (size_t ni = 0; ni < nodes.size(); ++ni) {
        const ConvNode &nd = nodes[ni];
        const int lay[2] = {nd.layer, nd.fused_layer};
        const isc_layer &L0 = layers[nd.layer].d;
        for (int k = 0; k < 2; ++k) {
            if (lay[k] < 0) continue;
            const isc_layer &L = layers[lay[k]].d;
            const int out_t = lay[k] + 1;
            PlanTensor &o = T[(size_t)out_t];
            // (a) in place over the residual operand, when this layer is its last reader
            if (L.res_tensor >= 0 && L.stride == 1 && T[(size_t)L.res_tensor].last_use_layer == lay[k] &&
                L.res_tensor != L.in_tensor && T[(size_t)L.res_tensor].halo == o.halo &&
                T[(size_t)L.res_tensor].bytes == o.bytes) {
                o.buffer = T[(size_t)L.res_tensor].buffer;
                continue;
            }
            // (b) over a same-shaped tensor whose last reader was the previous conv phase
            int reuse = -1;
            if (L.stride == 1 && lay[1] < 0 && prev_conv_layer_last >= 0)
                for (int t = 1; t <= n_conv_layers && reuse < 0; ++t) {
                    const PlanTensor &x = T[(size_t)t];
                    if (x.buffer < 0 || t == out_t || t == L.in_tensor || t == L.res_tensor) continue;
                    if (x.last_use_layer != prev_conv_layer_last) continue;
                    if (x.C != o.C || x.H != o.H || x.W != o.W || x.halo != o.halo) continue;
                    bool newest = true;           // x must be the current tenant of its buffer
                    for (int u = t + 1; u <= n_conv_layers; ++u)
                        if (T[(size_t)u].buffer == x.buffer) newest = false;
                    if (newest) reuse = x.buffer;
                }
            if (reuse >= 0) { o.buffer = reuse; continue; }
            new_buffer(out_t);
        }
        (void)L0;
        for (int k = 0; k < 2; ++k)
            if (lay[k] >= 0) layer_phase[(size_t)lay[k]] = (int)skel.size();
        skel.push_back({PH_CONV, (int)ni, -1});
        prev_conv_layer_last = nd.fused_layer >= 0 ? nd.fused_layer : nd.layer;
    }
    const int tail_phase = (int)skel.size();
    skel.push_back({PH_TAIL, -1, n_conv_layers});
    layer_phase[(size_t)n_layers - 2] = tail_phase;
    layer_phase[(size_t)n_layers - 1] = tail_phase;
    const int n_phases = (int)skel.size();
    if (n_phases > kMaxPhases || n_phases >= 256) return false;
    // ---- lifetimes
    for (int t = 0; t <= n_conv_layers; ++t) {
        PlanTensor &x = T[(size_t)t];
        if (x.buffer < 0) return false;
        int death = x.last_use_layer >= 0 ? layer_phase[(size_t)x.last_use_layer] : -1;
        if (t >= 1) x.producer_phase = layer_phase[(size_t)t - 1];
        else x.producer_phase = 1;
        death = std::max(death, x.producer_phase);
        buffers[(size_t)x.buffer].death = std::max(buffers[(size_t)x.buffer].death, death);
    }
    // ---- weight blobs: conv c is loaded when conv c-1 starts (conv 0 at the start of the group)
    std::vector<int> conv_phase;
    for (int ph = 0; ph < n_phases; ++ph)
        if (skel[(size_t)ph].kind == PH_CONV) conv_phase.push_back(ph);
    const int n_conv = (int)conv_phase.size();
    std::vector<uint32_t> w_bytes((size_t)n_conv), w_off((size_t)n_conv), n_rows((size_t)n_conv);
    std::vector<std::vector<std::pair<int, int>>> ksteps((size_t)n_conv);   // indices into chunk list, -1 = none
    std::vector<std::vector<int>> chunk_addr((size_t)n_conv);
    for (int cidx = 0; cidx < n_conv; ++cidx) {
        const ConvNode &nd = nodes[(size_t)skel[(size_t)conv_phase[(size_t)cidx]].node];
        const isc_layer &L = layers[nd.layer].d;
        const PlanTensor &in = T[(size_t)L.in_tensor];
        const int taps = L.kh * L.kw;
        std::vector<int> addr;
        for (int tap = 0; tap < taps; ++tap)
            for (int pl = 0; pl < in.planes; ++pl) {
                const int r = tap / L.kw, s = tap % L.kw;
                addr.push_back(((r - L.pad) * in.Wp + (s - L.pad)) * 16 + pl * (int)in.plane_bytes);
            }
        std::vector<std::pair<int, int>> ks;
        for (size_t a = 0; a < addr.size(); a += 2) {
            if (a + 1 < addr.size()) {
                if (addr[a + 1] > addr[a]) ks.push_back({(int)a, (int)a + 1});
                else ks.push_back({(int)a + 1, (int)a});
                const int diff = std::abs(addr[a + 1] - addr[a]);
                if (diff == 0 || diff >= (1 << 18)) return false;
            } else {
                ks.push_back({(int)a, -1});
            }
        }
        if ((int)ks.size() > kMaxKsteps) return false;
        ksteps[(size_t)cidx] = ks;
        chunk_addr[(size_t)cidx] = addr;
        n_rows[(size_t)cidx] = (uint32_t)(L.cout + (nd.fused_layer >= 0 ? layers[nd.fused_layer].d.cout : 0));
        w_bytes[(size_t)cidx] = (uint32_t)sizeof(ConvDesc) + (uint32_t)ks.size() * n_rows[(size_t)cidx] * 32u + n_rows[(size_t)cidx] * 16u;
    }
    // ---- shared-memory placement in order of birth
    std::vector<AllocReq> reqs, placed;
    for (PlanBuffer &b : buffers) reqs.push_back({b.bytes, b.birth, b.death, 0, &b.off});
    for (int cidx = 0; cidx < n_conv; ++cidx)
        reqs.push_back({w_bytes[(size_t)cidx], cidx == 0 ? 0 : conv_phase[(size_t)cidx - 1], conv_phase[(size_t)cidx],
                        cidx == 0 ? 0 : 1, &w_off[(size_t)cidx]});
    std::stable_sort(reqs.begin(), reqs.end(), [](const AllocReq &a, const AllocReq &b) { return a.birth < b.birth; });
    uint32_t high = kCtrlBytes;
    for (AllocReq &r : reqs) {
        if (!place(placed, r, kSmemLimit)) return false;
        high = std::max(high, *r.off + r.bytes);
    }
    // ---- emit phases
    plan->phases.assign((size_t)n_phases, MPhase{});
    plan->conv_phase = conv_phase;
    plan->tensors = T;
    plan->tensor_off.assign(T.size(), 0);
    for (int t = 0; t <= n_conv_layers; ++t) plan->tensor_off[(size_t)t] = buffers[(size_t)T[(size_t)t].buffer].off;
    int item_base = 0, round_base = 0, last_cols = -1;
    blob_out->clear();
    blob_offsets->assign((size_t)n_conv, 0);
    bool magic_ok = true;
    for (int ph = 0; ph < n_phases; ++ph) {
        MPhase &P = plan->phases[(size_t)ph];
        const Skel &S = skel[(size_t)ph];
        P.kind = S.kind;
        P.item_base = item_base;
        P.full_sync = 1;
        if (S.kind == PH_FILL) {
            const PlanTensor &x = T[(size_t)S.tensor];
            P.fill_off = plan->tensor_off[(size_t)S.tensor];
            P.fill_bytes = x.bytes;
            P.fill_word = (uint32_t)(x.halo & 0xFF) * 0x01010101u;
            P.n_items = (int)((x.bytes + kFillItemBytes - 1) / kFillItemBytes);
        } else if (S.kind == PH_INPUT) {
            const PlanTensor &x = T[0];
            if (x.W % 4 != 0) return false;
            P.H = x.H; P.W = x.W; P.Wp = x.Wp; P.HsWp = x.HsWp; P.P_first = x.P_first;
            P.n_items = (G * x.H * (x.W / 4) + 127) / 128;
        } else if (S.kind == PH_TAIL) {
            P.n_items = (G + 3) / 4;
        } else {
            const ConvNode &nd = nodes[(size_t)S.node];
            const int cidx = (int)(std::find(conv_phase.begin(), conv_phase.end(), ph) - conv_phase.begin());
            const isc_layer &L = layers[nd.layer].d;
            const PlanTensor &in = T[(size_t)L.in_tensor];
            P.H = in.H; P.W = in.W; P.Wp = in.Wp; P.HsWp = in.HsWp; P.P_first = in.P_first;
            P.n_tiles = in.n_tiles;
            P.magic_hswp = magic_for((uint32_t)in.HsWp, (uint32_t)in.npa + 256, &magic_ok);
            P.magic_wp = magic_for((uint32_t)in.Wp, (uint32_t)in.HsWp + 256, &magic_ok);
            P.scatter = L.stride == 2;
            const PlanTensor &o0 = T[(size_t)nd.layer + 1];
            P.o_Wp = o0.Wp; P.o_HsWp = o0.HsWp;
            P.in_off = plan->tensor_off[(size_t)L.in_tensor];
            P.n_ksteps = (uint32_t)ksteps[(size_t)cidx].size();
            P.n_rows = (int)n_rows[(size_t)cidx];
            P.n_chunks = n_rows[(size_t)cidx] / 16;
            if (P.n_chunks > kMaxChunks) return false;
            P.idesc = (2u << 4) | ((L.in_tensor == 0 ? 0u : 1u) << 7) | (1u << 10) |
                      ((uint32_t)(P.n_rows >> 3) << 17) | ((128u >> 4) << 24);
            P.w_off = w_off[(size_t)cidx];
            P.w_bytes = w_bytes[(size_t)cidx];
            const uint32_t weights_rel = (uint32_t)sizeof(ConvDesc);
            const uint32_t consts_rel = weights_rel + P.n_ksteps * (uint32_t)P.n_rows * 32u;
            P.const_off = P.w_off + consts_rel;
            P.conv_index = (uint32_t)cidx;
            // rounds: at most half of tensor memory each, at least two per phase so that the tensor cores work on
            // one half while the other is requantised, an even number of tiles in all but the last
            if (P.n_rows > kMaxFusedCols) return false;
            const int tile_cols = tile_columns(P.n_rows), per_half = kHalfCols / tile_cols;
            int n_rounds = std::max((in.n_tiles + per_half - 1) / per_half, in.n_tiles >= 2 ? 2 : 1);
            P.tiles_per_round = ((in.n_tiles + n_rounds - 1) / n_rounds + 1) & ~1;
            P.n_rounds = (in.n_tiles + P.tiles_per_round - 1) / P.tiles_per_round;
            if (P.tiles_per_round > per_half || P.n_rounds > 255) return false;
            P.n_items = P.n_rounds;
            round_base += P.n_rounds;
            for (uint32_t k = 0; k < P.n_ksteps; ++k) {
                const auto &kp = ksteps[(size_t)cidx][k];
                P.a_delta[k] = chunk_addr[(size_t)cidx][(size_t)kp.first];
                P.a_lbo[k] = kp.second >= 0 ? (uint32_t)(chunk_addr[(size_t)cidx][(size_t)kp.second] -
                                                         chunk_addr[(size_t)cidx][(size_t)kp.first]) : 16u;
            }
            // operand reads must stay inside the input region
            for (uint32_t k = 0; k < P.n_ksteps; ++k) {
                const long long lo_b = (long long)P.P_first * 16 + P.a_delta[k];
                const long long hi_b = (long long)(P.P_first + 128 * P.n_tiles) * 16 + P.a_delta[k] + P.a_lbo[k];
                if (lo_b < 0) return false;
                const long long plane_of_hi = (hi_b - 1) / in.plane_bytes;
                if (plane_of_hi >= in.planes) return false;
            }
            // dependencies: tile rule only when the operand was written, tile for tile, by the previous phase
            const bool prev_is_conv = ph >= 1 && skel[(size_t)ph - 1].kind == PH_CONV;
            bool tile_rule = prev_is_conv && in.producer_phase == ph - 1 && !in.scatter_produced;
            if (L.res_tensor >= 0 && T[(size_t)L.res_tensor].producer_phase >= ph - 1) tile_rule = false;
            if (tile_rule && plan->phases[(size_t)ph - 1].n_tiles != P.n_tiles) tile_rule = false;
            if (tile_cols != last_cols) tile_rule = false;   // rounds of another size: no round-for-round rule
            last_cols = tile_cols;
            P.full_sync = tile_rule ? 0 : 1;
            // epilogue chunks and the weight blob
            const int lay[2] = {nd.layer, nd.fused_layer};
            std::vector<uint8_t> blob(P.w_bytes, 0);
            int row0 = 0;
            int chunk = 0;
            for (int k2 = 0; k2 < 2; ++k2) {
                if (lay[k2] < 0) continue;
                const MegaLayerIn &ML = layers[lay[k2]];
                const isc_layer &LL = ML.d;
                PlanTensor &o = T[(size_t)lay[k2] + 1];
                o.scatter_produced = LL.stride == 2;
                plan->tensors[(size_t)lay[k2] + 1].scatter_produced = o.scatter_produced;
                const int taps = LL.kh * LL.kw;
                if (LL.res_tensor >= 0) {
                    P.res_mult = LL.res_mult;
                    P.res_n = 31 - LL.res_shift;
                    P.res_R = (1ll << (P.res_n - 1)) - (long long)LL.zp_res * LL.res_mult;
                }
                for (int pl = 0; pl < o.planes; ++pl, ++chunk) {
                    ChunkInfo &ci = P.chunk[chunk];
                    ci.out_off = plan->tensor_off[(size_t)lay[k2] + 1] + (uint32_t)pl * o.plane_bytes;
                    ci.res_off = LL.res_tensor >= 0
                        ? plan->tensor_off[(size_t)LL.res_tensor] + (uint32_t)pl * T[(size_t)LL.res_tensor].plane_bytes : 0u;
                    const int lo = LL.relu ? std::max(-128, LL.zp_out) : -128;
                    ci.lo = lo;
                    ci.halo = (uint32_t)(LL.zp_out & 0xFF) * 0x01010101u;
                    ci.flags = (lo > -128 ? 1u : 0u) | (LL.res_tensor >= 0 ? 2u : 0u);
                }
                for (int oc = 0; oc < LL.cout; ++oc) {
                    const int n = row0 + oc;
                    long long wsum = 0;
                    for (int q = 0; q < LL.cin * taps; ++q) wsum += ML.w[(size_t)oc * LL.cin * taps + q];
                    for (uint32_t k = 0; k < P.n_ksteps; ++k) {
                        const auto &kp = ksteps[(size_t)cidx][k];
                        const int halves[2] = {kp.first, kp.second};
                        for (int hf = 0; hf < 2; ++hf) {
                            if (halves[hf] < 0) continue;
                            const int tap = halves[hf] / in.planes, pl = halves[hf] % in.planes;
                            int src_tap = tap;
                            if (k2 == 1) {             // the 1x1 projection rides on the centre tap of the 3x3
                                if (tap != (L.kh / 2) * L.kw + L.kw / 2) continue;
                                src_tap = 0;
                            }
                            for (int b = 0; b < 16; ++b) {
                                const int ci = pl * 16 + b;
                                if (ci >= LL.cin) continue;
                                const int8_t wv = ML.w[((size_t)oc * LL.cin + ci) * taps + src_tap];
                                blob[weights_rel + (size_t)k * P.n_rows * 32 + (size_t)(n / 8) * 256 + (size_t)hf * 128 +
                                     (size_t)(n % 8) * 16 + b] = (uint8_t)wv;
                            }
                        }
                    }
                    const int sh = ML.shift[oc];
                    if (sh < 1 || sh > 20) return false;
                    const int nn = 31 + sh;
                    const long long biasf = (long long)ML.bias[oc] - (long long)LL.zp_in * wsum;
                    const long long B = biasf * ML.mult[oc] + (1ll << (nn - 1)) + ((long long)LL.zp_out << nn);
                    int32_t cst[4] = {(int32_t)(uint32_t)(B & 0xFFFFFFFFll), (int32_t)(B >> 32), ML.mult[oc], nn - 32};
                    memcpy(&blob[consts_rel + (size_t)n * 16], cst, 16);
                }
                row0 += LL.cout;
            }
            for (uint32_t q = 1; q < P.n_chunks; ++q)
                if (P.chunk[q].flags != P.chunk[0].flags) return false;      // one epilogue variant per phase
            ConvDesc D;
            memset(&D, 0, sizeof(D));
            D.in_off = P.in_off; D.n_ksteps = P.n_ksteps; D.idesc = P.idesc; D.n_rows = (uint32_t)P.n_rows;
            D.P_first = P.P_first; D.HsWp = P.HsWp; D.Wp = P.Wp; D.scatter = P.scatter;
            D.o_Wp = P.o_Wp; D.o_HsWp = P.o_HsWp; D.magic_hswp = P.magic_hswp; D.magic_wp = P.magic_wp;
            D.n_chunks = P.n_chunks; D.weights_rel = weights_rel; D.consts_rel = consts_rel;
            D.mode = (P.chunk[0].flags & 3u) | ((P.chunk[0].flags & 2u) && P.res_n >= 32 ? 4u : 0u);
            D.res_mult = P.res_mult; D.res_n = P.res_n; D.res_R = P.res_R;
            for (int q = 0; q < kMaxChunks; ++q) D.chunk[q] = P.chunk[q];
            for (int q = 0; q < kMaxKsteps; ++q) { D.a_delta[q] = P.a_delta[q]; D.a_lbo[q] = P.a_lbo[q]; }
            memcpy(blob.data(), &D, sizeof(D));
            (*blob_offsets)[(size_t)cidx] = (uint32_t)blob_out->size();
            blob_out->insert(blob_out->end(), blob.begin(), blob.end());
            while (blob_out->size() % 128) blob_out->push_back(0);
        }
        if (S.kind != PH_CONV) round_base += 1;
        item_base += P.n_items;
    }
    if (!magic_ok) return false;
    plan->G = G;
    plan->rounds_per_group = round_base;
    plan->smem_bytes = (high + 127u) & ~127u;
    return true;
}

}  // namespace

int mega_build(const MegaLayerIn *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes, MegaPlan **out)
{
    *out = nullptr;
    if (n_layers < 3 || n_classes > 128) return ISC_OK;
    // structure: convolutions, then global average pool, then FC
    const isc_layer &LP = layers[n_layers - 2].d, &LF = layers[n_layers - 1].d;
    if (LP.op != ISC_GAVGPOOL || LF.op != ISC_FC) return ISC_OK;
    if (LP.in_tensor != n_layers - 2 || LF.in_tensor != n_layers - 1) return ISC_OK;
    if (LP.cin > 64 || LP.cin % 16 != 0 || LF.res_tensor >= 0) return ISC_OK;
    for (int i = 0; i < n_layers - 2; ++i) {
        const isc_layer &L = layers[i].d;
        if (!conv_ok(L, i == 0)) return ISC_OK;
        if ((i == 0) != (L.in_tensor == 0)) return ISC_OK;
        if (L.res_tensor == 0) return ISC_OK;
        // a consumer's zero-point must be the halo value its operand was written with
        if (L.in_tensor > 0 && L.zp_in != layers[L.in_tensor - 1].d.zp_out) return ISC_OK;
        if (L.res_tensor > 0 && L.res_tensor > n_layers - 2) return ISC_OK;
    }
    if (LP.zp_in != layers[n_layers - 3].d.zp_out) return ISC_OK;
    for (int i = 1; i < n_layers - 2; ++i)
        if (layers[i].d.in_tensor > n_layers - 2) return ISC_OK;

    MegaPlan *plan = new MegaPlan();
    std::vector<uint8_t> blob;
    std::vector<uint32_t> blob_off;
    bool ok = false;
    for (int G = 4; G >= 1 && !ok; --G)
        ok = plan_for_G(layers, n_layers, in_c, in_h, in_w, n_classes, G, plan, &blob, &blob_off);
    if (!ok) { delete plan; return ISC_OK; }
    plan->in_c = in_c; plan->in_h = in_h; plan->in_w = in_w; plan->n_classes = n_classes;

    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        cudaGetLastError(); delete plan; return ISC_ERR_CUDA;
    }
    if (prop.major != 10 || (size_t)prop.sharedMemPerBlockOptin < plan->smem_bytes) { delete plan; return ISC_OK; }
    plan->sm_count = prop.multiProcessorCount;

    // FC parameters (bias folded with the pool output's zero-point)
    const int C = LP.cin;
    std::vector<int8_t> fcw((size_t)n_classes * 64, 0);
    std::vector<FcConst> fcc((size_t)n_classes);
    const MegaLayerIn &MF = layers[n_layers - 1];
    for (int o = 0; o < n_classes; ++o) {
        long long wsum = 0;
        for (int c = 0; c < C; ++c) {
            fcw[(size_t)o * 64 + c] = MF.w[(size_t)o * C + c];
            wsum += MF.w[(size_t)o * C + c];
        }
        FcConst k{};
        k.mult = MF.mult[o]; k.n = 31 + MF.shift[o]; k.zp_out = LF.zp_out;
        k.lo = LF.relu ? std::max(-128, LF.zp_out) : -128;
        k.bias = (int32_t)(MF.bias[o] - (long long)LF.zp_in * wsum);
        fcc[(size_t)o] = k;
    }
    bool cuda_ok = true;
    auto up = [&](void **dst, const void *src, size_t bytes) {
        if (cudaMalloc(dst, std::max<size_t>(bytes, 16)) != cudaSuccess) { cuda_ok = false; *dst = nullptr; return; }
        if (cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice) != cudaSuccess) cuda_ok = false;
    };
    up((void **)&plan->d_blob, blob.data(), blob.size());
    std::vector<PhaseEntry> ptab(plan->phases.size());
    for (size_t i = 0; i < ptab.size(); ++i) {
        const MPhase &P = plan->phases[i];
        ptab[i].kind_sync = (uint32_t)P.kind | ((uint32_t)(P.full_sync ? 1 : 0) << 8) |
                            (P.kind == PH_CONV ? (P.n_chunks << 16) : 0u);
        ptab[i].n_items = P.kind == PH_CONV ? (uint32_t)P.n_rounds | ((uint32_t)P.tiles_per_round << 8) |
                                                  ((uint32_t)tile_columns(P.n_rows) << 16)
                                            : (uint32_t)P.n_items;
        ptab[i].a = P.kind == PH_CONV ? P.w_off : P.fill_off;
        ptab[i].b = P.kind == PH_FILL ? (P.fill_bytes | ((P.fill_word & 0xFFu) << 24))
                                      : P.kind == PH_CONV ? (uint32_t)P.n_tiles : 0u;
    }
    std::vector<ConvSrc> csrc(plan->conv_phase.size());
    for (size_t c = 0; c < csrc.size(); ++c) {
        const MPhase &P = plan->phases[(size_t)plan->conv_phase[c]];
        csrc[c].gmem = (unsigned long long)(plan->d_blob + blob_off[c]);
        csrc[c].bytes_phase = P.w_bytes | ((uint32_t)plan->conv_phase[c] << 24);
        csrc[c].smem_off = P.w_off;
    }
    up((void **)&plan->d_ptab, ptab.data(), ptab.size() * sizeof(PhaseEntry));
    up((void **)&plan->d_conv_src, csrc.data(), csrc.size() * sizeof(ConvSrc));
    up((void **)&plan->d_fc_w, fcw.data(), fcw.size());
    up((void **)&plan->d_fc_c, fcc.data(), fcc.size() * sizeof(FcConst));
    int32_t zero = 0;
    up((void **)&plan->d_err, &zero, sizeof(zero));
    if (cuda_ok && cudaMalloc((void **)&plan->d_dump, kSmemLimit) != cudaSuccess) cuda_ok = false;
    if (!cuda_ok) { cudaGetLastError(); mega_free(plan); return ISC_ERR_NOMEM; }

    MegaParams &b = plan->base;
    memset(&b, 0, sizeof(b));
    b.ptab = plan->d_ptab;
    b.conv_src = plan->d_conv_src;
    b.in_H = plan->tensors[0].H; b.in_W = plan->tensors[0].W; b.in_Wp = plan->tensors[0].Wp; b.in_HsWp = plan->tensors[0].HsWp;
    b.n_phases = (int)plan->phases.size();
    b.n_conv = (int)plan->conv_phase.size();
    b.rounds_per_group = plan->rounds_per_group;
    b.G = plan->G;
    b.in_c = in_c;
    b.input_off = plan->tensor_off[0];
    b.input_halo = layers[0].d.zp_in;
    const PlanTensor &last = plan->tensors[(size_t)n_layers - 2];
    b.tail_in_off = plan->tensor_off[(size_t)n_layers - 2];
    b.tail_plane_bytes = last.plane_bytes;
    b.tail_C = last.C; b.tail_H = last.H; b.tail_W = last.W; b.tail_Wp = last.Wp; b.tail_HsWp = last.HsWp;
    b.pool_mult = layers[n_layers - 2].mult[0];
    b.pool_n = 31 + layers[n_layers - 2].shift[0];
    b.pool_zp_in = LP.zp_in; b.pool_zp_out = LP.zp_out;
    b.pool_lo = LP.relu ? std::max(-128, LP.zp_out) : -128;
    b.fc_w = plan->d_fc_w; b.fc_c = plan->d_fc_c;
    b.n_classes = n_classes;
    b.err = plan->d_err;
    b.stop_phase = 1 << 30;
    *out = plan;
    return ISC_OK;
}

void mega_free(MegaPlan *p)
{
    if (!p) return;
    cudaFree(p->d_ptab); cudaFree(p->d_conv_src); cudaFree(p->d_blob); cudaFree(p->d_fc_w);
    cudaFree(p->d_fc_c); cudaFree(p->d_err); cudaFree(p->d_dump);
    delete p;
}

static int mega_launch(MegaPlan *p, MegaParams &q, cudaStream_t st)
{
    if (!p->attr_set) {
        if (cudaFuncSetAttribute(k_mega, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p->smem_bytes) != cudaSuccess) {
            cudaGetLastError();
            return ISC_ERR_CUDA;
        }
        p->attr_set = true;
    }
    const int grid = std::max(1, std::min(q.n_groups, p->sm_count));
#ifdef ISC_TRACE
    {
        const char *lo = getenv("ISC_TRACE_LO"), *hi = getenv("ISC_TRACE_HI");
        const unsigned vlo = lo ? (unsigned)atoi(lo) : 0u, vhi = hi ? (unsigned)atoi(hi) : 0u, zero = 0u;
        cudaMemcpyToSymbol(g_trace_lo, &vlo, sizeof(vlo));
        cudaMemcpyToSymbol(g_trace_hi, &vhi, sizeof(vhi));
        cudaMemcpyToSymbol(g_trace_n, &zero, sizeof(zero));
    }
#endif
    k_mega<<<grid, kThreads, p->smem_bytes, st>>>(q);
    return cudaGetLastError() == cudaSuccess ? ISC_OK : ISC_ERR_CUDA;
}

int mega_run(MegaPlan *p, const uint8_t *d_x, const NoiseStream &ns, int64_t n, int batch_hint, int32_t *d_counts,
             int8_t *d_logits, cudaStream_t st, int64_t *launches)
{
    const int64_t per_launch = batch_hint > 0 ? batch_hint : (1ll << 30);
    for (int64_t done = 0; done < n; done += per_launch) {
        const int64_t m = std::min(per_launch, n - done);
        MegaParams q = p->base;
        q.x = d_x;
        q.ns = ns;
        q.ns.first_sample = ns.first_sample + done;
        q.n_samples = (int32_t)m;
        q.n_groups = (int32_t)((m + p->G - 1) / p->G);
        q.counts = d_counts;
        q.logits = d_logits ? d_logits + (size_t)done * p->n_classes : nullptr;
        int rc = mega_launch(p, q, st);
        *launches += 1;
        if (rc) return rc;
    }
    return ISC_OK;
}

int mega_check(MegaPlan *p)
{
    int32_t e = 0;
    if (cudaMemcpy(&e, p->d_err, sizeof(e), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return ISC_ERR_CUDA; }
    if (e != 0) {
        cudaMemset(p->d_err, 0, sizeof(e));
        return ISC_ERR_TIMEOUT;
    }
    return ISC_OK;
}

int mega_tensor_phase(MegaPlan *p, int tensor)
{
    if (tensor < 0 || tensor >= (int)p->tensors.size() || p->tensors[(size_t)tensor].buffer < 0) return -1;
    return p->tensors[(size_t)tensor].producer_phase;
}

// Runs one group (samples ns.first_sample ..) up to the phase that produces `tensor` and returns that
// tensor of the first sample as [C][H][W] int32.
int mega_debug_tensor(MegaPlan *p, const uint8_t *d_x, const NoiseStream &ns, int tensor, int32_t *out_chw,
                      int32_t *d_counts_scratch, cudaStream_t st, int64_t *launches)
{
    const int ph = mega_tensor_phase(p, tensor);
    if (ph < 0) return ISC_ERR_UNSUPPORTED;
    const PlanTensor &t = p->tensors[(size_t)tensor];
    MegaParams q = p->base;
    q.x = d_x; q.ns = ns; q.n_samples = 1; q.n_groups = 1; q.counts = d_counts_scratch; q.logits = nullptr;
    q.stop_phase = ph;
    q.dump_off = p->tensor_off[(size_t)tensor]; q.dump_bytes = t.bytes; q.dump = p->d_dump;
    int rc = mega_launch(p, q, st);
    *launches += 1;
    if (rc) return rc;
    std::vector<uint8_t> h(t.bytes);
    if (cudaMemcpyAsync(h.data(), p->d_dump, t.bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ISC_ERR_CUDA; }
    if ((rc = mega_check(p))) return rc;
    for (int c = 0; c < t.C; ++c)
        for (int y = 0; y < t.H; ++y)
            for (int x = 0; x < t.W; ++x) {
                const size_t pos = (size_t)(y + 1) * t.Wp + x + 1;
                const uint8_t b = h[(size_t)(c / 16) * t.plane_bytes + pos * 16 + (c % 16)];
                out_chw[((size_t)c * t.H + y) * t.W + x] = tensor == 0 ? (int32_t)b : (int32_t)(int8_t)b;
            }
    return ISC_OK;
}

#ifdef ISC_TRACE
// Copies the recorded triples to the host; returns how many there are.
extern "C" int isc_trace_read(unsigned long long *out, int max_events)
{
    unsigned n = 0;
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(&n, g_trace_n, sizeof(n));
    n = std::min(n, std::min(kTraceMax, (unsigned)max_events));
    cudaMemcpyFromSymbol(out, g_trace, (size_t)n * 3 * sizeof(unsigned long long));
    return (int)n;
}
#endif

}  // namespace isc
