// Line-tiled shared-memory-resident tensor-core engine (sm_100a) for CIFAR-shaped residual networks.
//
// One persistent CTA per SM carries a group of four noisy samples through the whole network.  Activations
// stay in shared memory, every convolution is an implicit GEMM on tcgen05 (kind::i8, int32 accumulators in
// tensor memory) and only vote counts return to global memory (Algorithm 1 steps 1-4, Algorithm 2 steps 1-2).
//
// Layout.  A tensor of C channels and H x W pixels (W = 32, 16 or 8) is stored per plane of 16 channels as
// "lines" of 128 positions of 16 bytes.  Position x * I + b * 4 + s of line l holds pixel (row l + b * L, column x)
// of sample s, where I = 128 / W positions belong to one column, I / 4 row bands b share a line and L = H / (I / 4)
// is the number of lines.  Lines are I positions apart from each other (a gap that always holds the zero-point:
// the left and right padding of every row), there is one more line above and below (the padding rows of the
// first and last band; for the other bands these two lines hold copies of the neighbouring band's edge rows,
// written together with the originals), so
//   * the horizontal neighbours of all 128 positions of a line are the same 128 positions moved by +-I, and
//   * the vertical neighbours of all 128 positions of line l are the same 128 positions of line l +- 1.
// A line is therefore an M = 128 operand tile whose nine filter taps are plain address offsets, with every one
// of its rows a real output pixel.
//
// Stacked convolutions.  For a 3x3, stride-1 convolution the three vertical taps are stacked along N: one MMA
// chain over input line p (K = three horizontal taps x input channels) accumulates into the accumulator
// columns of output lines p-1, p, p+1 at once (N = 3 x cout), because the accumulators of consecutive output
// lines are consecutive column blocks of tensor memory.  The epilogue zeroes a line's columns after reading
// them.  This triples N for the small channel counts where an MMA is bound by fetching its 128 x 32-byte A
// operand.  Strided and 1x1 convolutions, and those with cout = 64, run unstacked: one chain per output line
// over all taps.
//
// Roles.  Three issuing warps (lane 0 of each) share the MMA chains of a convolution: the host prepares a table of
// operations (accumulator columns, descriptor offsets, which units of the previous convolution must be stored,
// which units complete) in the order in which their inputs become available; operation i belongs to issuing warp
// i mod 3.  One thread alone cannot feed the tensor pipe: an MMA costs it about a hundred cycles of issue latency and
// a commit as much again, so the loop is kept to the fewest instructions (dependency counters read together, the
// timed wait out of line).  Sixteen epilogue warps requantise: four sets of four warps (one per 32-lane quarter of
// tensor memory) share the items of a convolution, an item being one unit (two or four output lines: one
// "accumulators complete" barrier pair, one "stored" counter) and one 16-channel chunk, in the order in which they
// complete.  The requantisation is integer arithmetic on a pipe that issues multiplies, shifts and packs at half
// rate: the pass is written for the fewest such instructions (see ChanConst4).  A loader warp copies the next
// convolution's blob once its place is free.  Consecutive convolutions overlap unit by unit.  Input noise (Def. 3.3,
// Eq. 2; Def. 3.4), halo fills and the pool / FC / argmax tail are CTA-wide phases between barriers.
//
// Every device-side wait is bounded by a wall-clock limit; on expiry the CTA raises an abort flag, all
// remaining waits fall through, and the host reports ISC_ERR_TIMEOUT.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <vector>

#include "isc_line.h"
#include "isc_tc.cuh"

namespace isc {

using namespace tc;

namespace {

constexpr int kG = 4;                       // samples per group
constexpr int kEpiWarps = 16;               // the first warps: epilogue; set = warp / 4, tensor-memory quarter = warp % 4
constexpr int kSets = kEpiWarps / 4;
constexpr int kIssuers = 3;                 // the next warps: lane 0 of each issues every kIssuers-th MMA chain of a convolution
constexpr int kLoaderWarp = kEpiWarps + kIssuers;   // the last warp: weight copies
constexpr int kThreads = 32 * (kEpiWarps + kIssuers + 1);
constexpr int kMaxKsteps = 18;
constexpr int kMaxPhases = 160;
constexpr int kMaxBars = 128;
constexpr int kMaxLines = 32;               // output lines of one convolution
constexpr int kCtrlBytes = 10240;
constexpr int kMaxConv = 128;
constexpr int kSmemLimit = 227 * 1024;
constexpr int kTmemCols = 512;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait

enum { PH_FILL = 0, PH_INPUT = 1, PH_CONV = 2, PH_TAIL = 3 };
enum { ERR_NONE = 0, ERR_WAIT_DONE = 1, ERR_WAIT_WEIGHTS = 2, ERR_WAIT_READY = 3, ERR_WAIT_FULL = 4, ERR_WAIT_DRAIN = 5 };
enum { CF_STACKED = 1, CF_RES = 2, CF_LO = 4, CF_SCATTER = 8, CF_GENERAL = 16, CF_RSHORT = 32 };     // CF_GENERAL: the pass that decides everything at run time; CF_RSHORT: residual term without the 64-bit addend
// OPF_WAIT_ALL: every unit of the previous convolution; OPF_NULL: no MMAs, arrivals only; OPF_WAITS / OPF_WAITS4: the
// record names counters to test (two / four slots in use); bits 4-6: how many of them are distinct; bits 8-9: arrivals
enum { OPF_WAIT_ALL = 1, OPF_WAITS = 2, OPF_NULL = 4, OPF_WAITS4 = 8 };

// ---- what the kernel reads -------------------------------------------------------------------

// One entry per phase, copied to shared memory when the kernel starts.
//   CONV: a = shared-memory offset of the blob      FILL: a = offset, b = bytes, c = halo byte
struct alignas(16) PhaseEntry { uint32_t kind, a, b, c; };

// Where the blob of convolution c comes from (global) and goes to (shared).
// and which convolution must be complete before the copy may start: the counters stored[dep_first .. + dep_units)
// must have reached dep_mult * (group * dep_uses + dep_local + 1); dep_units = 0: nothing to wait for.
struct alignas(16) ConvSrc {
    unsigned long long gmem;
    uint32_t bytes_phase, smem_off;                 // bytes | phase << 24; offset | late << 31
    uint32_t dep_first, dep_units, dep_mult, dep_local_uses;     // dep_local | dep_uses << 16
};

// One MMA chain in the form the issuing thread consumes: accumulator columns, what to add to the operand
// descriptors' start addresses, and the barriers (as byte offsets, 0xFFFF = none) of its dependencies and completions.
struct alignas(16) LOp {
    uint32_t d_col;         // first accumulator column within the bank
    uint32_t idesc;         // instruction descriptor (N = blocks * cout)
    uint32_t a_add, b_add;  // 16-byte units: (input line + 1) * pitch, first weight block * block size
    uint16_t wait[4];       // 8 * unit of the previous convolution that must be stored
    uint16_t commit[3];     // 8 * unit of this convolution whose accumulators are complete after the chain
    uint16_t flags;         // OPF_* | distinct waits << 4 | arrivals << 8
};
static_assert(sizeof(LOp) == 32, "one operation is two 16-byte loads");

// Head of every blob: everything the issuing thread and the epilogue need to know about the convolution.
struct alignas(16) LConvDesc {
    uint32_t n_ops, n_passes, n_ksteps, flags;
    uint32_t a_base, pitch16, bblock16, n_banks;            // a_base: line -1, lane 0, plane 0 of the input
    uint32_t idesc[3], cols;                                // instruction descriptors for 1, 2, 3 blocks; columns per line
    uint32_t d_base[2], bar_full, bar_done;                 // accumulator bank bases; barrier indices of this class
    uint32_t use_local, uses_per_group, n_lines, n_chunks;
    uint32_t w_rel, c_rel, ops_rel, passes_rel;
    // epilogue: where results go (line 0, lane 0, plane 0), geometry of the output and of the scattered input
    uint32_t out_base, out_plane, out_pitch16, out_n_lines;
    uint32_t out_log_lines, out_nb, out_logI, res_base;
    uint32_t res_plane, in_logI, in_I, in_n_lines;
    int32_t lo; uint32_t res_m2, res_r2_lo, res_r2_hi;
    uint32_t b_lo0, kstep16, recs_per_item, pad1;       // low word of the first K-step's weight descriptor (shared-memory base 0); records per (unit, chunk)
    uint32_t a_lo[kMaxKsteps + 2];             // low words of the operand descriptors of line -1 (shared-memory base 0)
};
static_assert(sizeof(LConvDesc) % 16 == 0, "blob sections stay 16-byte aligned");

struct FcConst { int32_t mult, n, zp_out, lo, bias, pad0, pad1, pad2; };

struct LineParams {
    const PhaseEntry *ptab;
    const ConvSrc *conv_src;
    const uint8_t *bar_counts;
    int32_t n_bars, n_phases, n_conv, n_groups;
    int32_t n_samples, in_c, in_H, in_W;
    const uint8_t *x;                 // clean image, CHW
    NoiseStream ns;
    uint32_t input_base, input_pitch16;   // line 0, lane 0 of the first layer's operand region
    // tail
    uint32_t tail_base, tail_plane, tail_pitch16, tail_logI;
    int32_t tail_C, tail_H, tail_W, tail_n_lines;
    int32_t pool_mult, pool_n, pool_zp_in, pool_zp_out, pool_lo;
    const int8_t *fc_w;               // [n_classes][64]
    const FcConst *fc_c;
    int32_t n_classes;
    int32_t *counts;
    int8_t *logits;                   // [n_samples][n_classes] or null
    int32_t *err;
    unsigned long long *phase_cycles; // [4]: SM cycles per CTA spent in FILL, INPUT, everything else, TAIL, summed over CTAs and launches
    // debug
    int32_t stop_phase;
    uint32_t dump_off, dump_bytes;
    uint8_t *dump;
};

struct Ctrl {
    unsigned long long bars[kMaxBars];
    unsigned long long wbar[3], drain;
    uint32_t tmem_base;
    volatile int abort_flag;
    uint32_t stored[kMaxBars];              // per unit: stores of its 16-channel chunks by a warp, counted over the whole run
    int32_t hist[128];
    int32_t pooled[kG][64];                 // the tail's pooled features, one row per sample of the group
    long long cyc[4], cyc_mark;             // thread 0's phase clocks
    PhaseEntry ptab[kMaxPhases];
    ConvSrc csrc[kMaxConv];
};
static_assert(sizeof(Ctrl) <= kCtrlBytes - 16, "control block too large");

// ------------------------------------------------------------------ device helpers

__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void commit_to(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_st16_zero(uint32_t taddr)
{
    const int z = 0;
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
                 ::"r"(taddr), "r"(z) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ long long mad_wide_u(uint32_t a, uint32_t b, long long c)
{
    long long d;
    asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(d) : "r"(a), "r"(b), "l"(c));
    return d;
}
// Per-channel requantisation constants as stored in the blob (16 bytes): folded bias, multiplier, rounding addend
// and shift.  With s = shift - 1 >= 1,
//   rs((acc + bias) * mult, 31 + shift) + zp_out = (hi32((acc + bias) * mult) + c) >> s,   c = 2^(s-1) + zp_out * 2^s,
// exactly: the rounding half 2^(31+s) is a multiple of 2^32, so the low word of the product cannot change the floor.
// For s = 0 the half sits in the low word: the result is hi32 + (bit 31 of the low word) + c with c = zp_out.
// The integer pipe issues multiplies, shifts and packs at half rate here, a 64-bit addend costs two more
// instructions: this form is the cheapest exact one found (add, wide multiply, add, shift).
struct ChanConst4 { int bias, mult, c, s; };
// A plain load (the blob is complete in shared memory; the address derives from a value read after the wait for it)
// that the compiler may schedule ahead of the tensor-memory wait.
__device__ __forceinline__ ChanConst4 ld_chan_const_early(uint32_t addr)
{
    ChanConst4 c;
    asm("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(c.bias), "=r"(c.mult), "=r"(c.c), "=r"(c.s) : "r"(addr));
    return c;
}
__device__ __forceinline__ long long mul_wide(int a, int b)
{
    long long d;
    asm("mul.wide.s32 %0, %1, %2;" : "=l"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ void red_release_add(uint32_t addr, uint32_t v)
{
    asm volatile("red.release.cta.shared::cta.add.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_volatile_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.volatile.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_acquire_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
// byte K of w, zero-extended
template <int K>
__device__ __forceinline__ uint32_t ubyte(uint32_t w)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, 0, %2;" : "=r"(d) : "r"(w), "n"(0x4440 | K));
    return d;
}

struct Waiter {
    Ctrl *ctrl;
    int32_t *err;
    unsigned long long limit_ns = kWaitLimitNs;
    __device__ __forceinline__ bool aborted() const { return ctrl->abort_flag != 0; }
    // the error word: wait kind | index of the barrier within the control block << 8 | parity waited for << 20 | CTA << 21
    __device__ __noinline__ void fail(int code, uint32_t bar, uint32_t parity)
    {
        ctrl->abort_flag = 1;
        const uint32_t idx = (bar - smem_u32(ctrl)) >> 3;
        atomicCAS(err, 0, (int)((uint32_t)code | ((idx & 0xFFFu) << 8) | ((parity & 1u) << 20) | (blockIdx.x << 21)));
    }
    // Wait for a phase of an mbarrier.  Each attempt parks the thread in hardware for a bounded time,
    // so a waiting warp does not compete for issue slots.
    __device__ __forceinline__ bool barrier(uint32_t bar, uint32_t parity, int code)
    {
        if (mbar_test(bar, parity)) return true;
        if (mbar_try(bar, parity)) return true;         // parks the thread; the clock is read only when this gives up
        const unsigned long long t0 = globaltimer();
        for (int spin = 0;; ++spin) {
            if (mbar_try(bar, parity)) return true;
            if ((spin & 7) == 7) {
                if (aborted()) return false;
                if (globaltimer() - t0 > limit_ns) { fail(code, bar, parity); return false; }
            }
        }
    }
    // Wait until a counter in shared memory has reached `expected` (counters only grow).
    __device__ __forceinline__ bool counter(uint32_t addr, uint32_t expected, int code)
    {
        // The first test is a plain load: an acquiring one costs over a hundred cycles here.  What the counter guards
        // was made visible to the tensor cores' reads by the storing warp (proxy fence, then a releasing add) and is
        // read by MMAs that are issued only after the value has been seen.
        if ((int32_t)(ld_volatile_u32(addr) - expected) >= 0) return true;
        const unsigned long long t0 = globaltimer();
        for (int spin = 0;; ++spin) {
            if ((int32_t)(ld_acquire_u32(addr) - expected) >= 0) return true;
            if ((spin & 15) == 15) {
                if (aborted()) return false;
                if (globaltimer() - t0 > limit_ns) { fail(code, addr, 0); return false; }
            }
        }
    }
};

// ------------------------------------------------------------------ issuing thread

struct PrevConv { uint32_t done_addr, expected, n_lines; };    // counters of its units, their value when stored; n_lines = 0: nothing to wait for

struct IssueCtx {
    uint32_t desc, ops, n_ops, s16, b_lo0, kstep16, d0, stacked, full_addr, cg, issuer;
};

// The first, cheap read of a "stored" counter by an issuing thread.  A plain load by default: an acquiring one costs
// over a hundred cycles per test on the issue path.  What the counter guards was published by the storing warp with a
// proxy fence and a releasing add; the MMAs that read it are issued after the value was seen (control dependency)
// and after tcgen05.fence::after_thread_sync.  Building with -DISC_ACQUIRE_POLL takes the acquiring form instead, so
// that a divergence could be traced to this choice.
__device__ __forceinline__ uint32_t ld_counter(uint32_t addr)
{
#ifdef ISC_ACQUIRE_POLL
    return ld_acquire_u32(addr);
#else
    return lds32(addr);
#endif
}

// The dependency test of an operation when its first, cheap form did not pass (or the operation waits for the whole
// previous convolution): bounded waits on every counter the record names.  Kept out of line: the issue loop is
// latency-bound, every instruction on its path counts.
__device__ __noinline__ bool wait_units_slow(Waiter w, const PrevConv &prev, uint4 r1)
{
    const uint32_t fl = r1.w >> 16;
    if (fl & OPF_WAIT_ALL)
        for (uint32_t l = 0; l < prev.n_lines; ++l)
            if (!w.counter(prev.done_addr + 4 * l, prev.expected, ERR_WAIT_DONE)) return false;
    const uint32_t nw = (fl >> 4) & 7u;
    const uint32_t off[4] = {r1.x & 0xFFFFu, r1.x >> 16, r1.y & 0xFFFFu, r1.y >> 16};
#pragma unroll
    for (uint32_t k = 0; k < 4; ++k)
        if (k < nw && !w.counter(prev.done_addr + off[k], prev.expected, ERR_WAIT_DONE)) return false;
    return true;
}

// The operations of one convolution that belong to one issuing thread (every kIssuers-th record).  The low words of
// the operand descriptors stay in registers; an operation adds its line and block offsets to their start-address
// fields.  The counters an operation depends on are read together (unused slots repeat the first one) and compared
// once; what the counters guard was made visible to the tensor cores' reads by the storing warp (proxy fence, then a
// releasing add) and is read by MMAs that are issued only after the values have been seen.
template <int KS>
__device__ __forceinline__ bool issue_ops(Waiter w, const IssueCtx &ic, const PrevConv &prev, uint32_t n_ksteps)
{
    constexpr int NK = KS > 0 ? KS : 1;
    uint32_t alo[NK], blo[NK];
    const uint32_t ahi = (uint32_t)(make_desc(0, 0, 128) >> 32), bhi = (uint32_t)(make_desc(0, 128, 256) >> 32);
    if (KS > 0) {
#pragma unroll
        for (int k4 = 0; k4 < NK; k4 += 4) {
            const uint4 v = ld_shared_v4(ic.desc + offsetof(LConvDesc, a_lo) + 4 * k4);
            const uint32_t vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (k4 + q < NK) alo[k4 + q] = vv[q] + ic.s16;
        }
#pragma unroll
        for (int k = 0; k < NK; ++k) blo[k] = ic.b_lo0 + ic.s16 + (uint32_t)k * ic.kstep16;
    }
    uint32_t at = ic.ops + 32u * ic.issuer;           // the table ends with kIssuers spare records: reads run one ahead
    uint4 n0 = ld_shared_v4(at), n1 = ld_shared_v4(at + 16);
    const uint32_t acc_first = ic.stacked;
    for (uint32_t i = ic.issuer; i < ic.n_ops; i += kIssuers) {
        const uint4 r0 = n0, r1 = n1;         // d_col, idesc, a_add, b_add | wait 0-1, wait 2-3, commit 0-1, commit 2 and flags
        at += 32u * kIssuers;
        n0 = ld_shared_v4(at); n1 = ld_shared_v4(at + 16);
        const uint32_t fl = r1.w >> 16;
        // units of the previous convolution this operation depends on
        if (fl & (OPF_WAIT_ALL | OPF_WAITS)) {
            int32_t m = -1;
            if (!(fl & OPF_WAIT_ALL)) {
                m = min((int32_t)(ld_counter(prev.done_addr + (r1.x & 0xFFFFu)) - prev.expected),
                        (int32_t)(ld_counter(prev.done_addr + (r1.x >> 16)) - prev.expected));
                if (fl & OPF_WAITS4)
                    m = min(m, min((int32_t)(ld_counter(prev.done_addr + (r1.y & 0xFFFFu)) - prev.expected),
                                   (int32_t)(ld_counter(prev.done_addr + (r1.y >> 16)) - prev.expected)));
            }
            if (m < 0 && !wait_units_slow(w, prev, r1)) return false;
        }
        tc_fence_after();
        const uint32_t d = ic.d0 + r0.x;
        if (fl & OPF_NULL) {
            // a record that only carries this thread's arrivals on units it did not add to
        } else if (KS > 0) {
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                const uint64_t ad = ((uint64_t)ahi << 32) | (uint64_t)(alo[k] + r0.z);
                const uint64_t bd = ((uint64_t)bhi << 32) | (uint64_t)(blo[k] + r0.w);
                mma_i8(d, ad, bd, r0.y, k > 0 ? 1u : acc_first);
            }
        } else {
            for (uint32_t k = 0; k < n_ksteps; ++k) {
                const uint32_t a_lo = lds32(ic.desc + offsetof(LConvDesc, a_lo) + 4 * k) + ic.s16;
                const uint64_t ad = ((uint64_t)ahi << 32) | (uint64_t)(a_lo + r0.z);
                const uint64_t bd = ((uint64_t)bhi << 32) | (uint64_t)(ic.b_lo0 + ic.s16 + k * ic.kstep16 + r0.w);
                mma_i8(d, ad, bd, r0.y, k > 0 ? 1u : acc_first);
            }
        }
        const uint32_t nc = (fl >> 8) & 3u;
        if (nc) {
            commit_to(ic.full_addr + (r1.z & 0xFFFFu));
            if (nc > 1) {
                commit_to(ic.full_addr + (r1.z >> 16));
                if (nc > 2) commit_to(ic.full_addr + (r1.w & 0xFFFFu));
            }
        }
    }
    return true;
}

__device__ __forceinline__ void issue_weights(const ConvSrc *src, uint32_t sbase, uint32_t wbar_addr)
{
    const uint4 v = *reinterpret_cast<const uint4 *>(src);
    const void *gmem = reinterpret_cast<const void *>(((unsigned long long)v.y << 32) | v.x);
    const uint32_t bytes = v.z & 0xFFFFFFu;
    mbar_expect_tx(wbar_addr, bytes);
    bulk_g2s(sbase + (v.w & 0x7FFFFFFFu), gmem, bytes, wbar_addr);
}

// The copy of convolution `target`'s blob, by lane 0 of the loader warp, once the convolution it names is complete:
// the blob takes the place of things that convolution (or an earlier one) was the last to use.
__device__ __noinline__ bool loader_copy(const LineParams &p, Ctrl *ctrl, uint32_t sbase, int target, uint32_t cg_target, int it)
{
    Waiter w{ctrl, p.err};
    const ConvSrc *src = ctrl->csrc + target;
    if ((int)(src->bytes_phase >> 24) > p.stop_phase) return true;
    const uint32_t n = src->dep_units;
    if (n) {
        const uint32_t expected = src->dep_mult * ((uint32_t)it * (src->dep_local_uses >> 16) + (src->dep_local_uses & 0xFFFFu) + 1u);
        const uint32_t first = smem_u32(&ctrl->stored[src->dep_first]);
        for (uint32_t l = 0; l < n; ++l)
            if (!w.counter(first + 4 * l, expected, ERR_WAIT_DONE)) return false;
    }
    issue_weights(src, sbase, smem_u32(&ctrl->wbar[cg_target % 3]));
    return true;
}

// One convolution's share of an issuing warp, by its lane 0.  Returns false after a wait has expired.
__device__ __noinline__ bool issuer_conv(const LineParams &p, Ctrl *ctrl, uint32_t sbase, uint32_t tmem, uint32_t blob_off,
                                         uint32_t cg, int issuer, int it, PrevConv &prev)
{
    Waiter w{ctrl, p.err};
    if (!w.barrier(smem_u32(&ctrl->wbar[cg % 3]), (cg / 3) & 1, ERR_WAIT_WEIGHTS)) return false;
    const uint32_t desc = sbase + blob_off;
    const uint4 h0 = ld_shared_v4(desc);                                    // n_ops, n_passes, n_ksteps, flags
    const uint4 h1 = ld_shared_v4(desc + offsetof(LConvDesc, a_base));      // a_base, pitch16, bblock16, n_banks
    const uint4 h3 = ld_shared_v4(desc + offsetof(LConvDesc, d_base));      // d_base[2], bar_full, bar_done
    const uint4 h4 = ld_shared_v4(desc + offsetof(LConvDesc, use_local));   // use_local, uses_per_group, n_lines, n_chunks
    const uint4 h5 = ld_shared_v4(desc + offsetof(LConvDesc, w_rel));       // w_rel, c_rel, ops_rel, passes_rel
    const uint4 hb = ld_shared_v4(desc + offsetof(LConvDesc, b_lo0));       // b_lo0, kstep16
    const uint32_t use = (uint32_t)it * h4.y + h4.x;
    IssueCtx ic;
    ic.desc = desc; ic.ops = desc + h5.z; ic.n_ops = h0.x;
    ic.s16 = sbase >> 4; ic.b_lo0 = hb.x; ic.kstep16 = hb.y;
    ic.d0 = tmem + ((h1.w > 1 && (use & 1u)) ? h3.y : h3.x);
    ic.stacked = (h0.w & CF_STACKED) ? 1u : 0u;
    ic.full_addr = smem_u32(&ctrl->bars[h3.z + (use & 1u) * h4.z]);      // the class has two sets of barriers, used in turn
    ic.cg = cg;
    ic.issuer = (uint32_t)issuer;
    bool ok;
    switch (h0.z) {
    case 1: ok = issue_ops<1>(w, ic, prev, 1); break;
    case 2: ok = issue_ops<2>(w, ic, prev, 2); break;
    case 3: ok = issue_ops<3>(w, ic, prev, 3); break;
    case 5: ok = issue_ops<5>(w, ic, prev, 5); break;
    case 9: ok = issue_ops<9>(w, ic, prev, 9); break;
    case 18: ok = issue_ops<18>(w, ic, prev, 18); break;
    default: ok = issue_ops<0>(w, ic, prev, h0.z); break;
    }
    if (!ok) return false;
    prev.done_addr = smem_u32(&ctrl->stored[h3.w]);
    prev.expected = 4u * h4.w * (use + 1u);
    prev.n_lines = h4.z;
    return true;
}

// ------------------------------------------------------------------ epilogue warps

struct EpiCtx {
    Ctrl *ctrl;
    uint32_t sbase, tmem_lane;          // tensor-memory address of this warp's 32 lanes, column 0
    int warp, set, quarter, lane, tid;
    uint32_t lane_idx;                  // position within a line: quarter * 32 + lane
};

// What an epilogue warp keeps in registers for the whole of a convolution: addresses already specialised to the
// thread (its position within a line, its 32 lanes of tensor memory), so that a pass only adds the offsets of its
// table record.  The geometry that only strided convolutions need stays in the blob's header.
struct EpiConv {
    uint32_t tmem0;                       // tensor-memory address of this warp's lanes, first column of the bank
    uint32_t full_addr, done_addr, parity;
    uint32_t const_addr;
    uint32_t out_thread, res_thread;      // line 0, this thread's position, plane 0 of the output / residual
    uint32_t dup_delta;                   // bytes from a band's first row to its copy below the band above; 0: one band
    uint32_t dup_up, dup_dn;              // this thread's band has a band above / below
    uint32_t res_m2;
    long long res_r2;
};

// One pass of the table: lines (a unit), chunk, and the offsets they imply.
struct alignas(16) LPass {
    uint32_t meta;          // unit | lines << 8 | chunk << 12 | line 0 first / last row of its band << 16, 17 | line 1 << 18, 19
    uint32_t lines;         // line 0 | line 1 << 8
    uint32_t tcol[2];       // accumulator columns of the two lines' chunk within the bank
    uint32_t out[2];        // byte offset of the two lines' chunk (line within its plane + plane) in the output
    uint32_t res[2];        // the same in the residual operand
};
static_assert(sizeof(LPass) == 32, "one pass is two 16-byte loads");

// One output of the common pass (every channel has s >= 1).
//   residual: y += floor((u * m2 + R2) / 2^32) with u = r + 128 the residual byte as an unsigned number,
//   m2 = res_mult * 2^(32-n) and R2 the rounding half and the zero-points folded: rs((r - zp_res) * res_mult, n).
//   kRes = 2: the same term as hi32((256 k + u) * m2) - c_r, for an offset k that the planner has checked on all 256
//   values of u (residual_short_form): `res_r2` then holds 256 k, which the byte permute that extracts u merges
//   into it, and c_r is folded into the channel's rounding addend.
template <int kRes, int K>
__device__ __forceinline__ int requant1(int acc, const ChanConst4 &cs, uint32_t rword, uint32_t res_m2, long long res_r2)
{
    int y = (hi32(mul_wide(acc + cs.bias, cs.mult)) + cs.c) >> cs.s;
    if (kRes == 1) y += hi32(mad_wide_u(ubyte<K>(rword), res_m2, res_r2));
    if (kRes == 2) {
        uint32_t u;
        asm("prmt.b32 %0, %1, %2, %3;" : "=r"(u) : "r"(rword), "r"((uint32_t)lo32(res_r2)), "n"(0x7650 | K));
        y += hi32(mad_wide_u(u, res_m2, 0ll));
    }
    return y;
}

__device__ __forceinline__ void st_shared_v4_if(uint32_t addr, uint4 v, uint32_t flag)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %5, 0;\n\t@p st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n\t}"
                 ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(flag) : "memory");
}

// The wait of a pass for its unit's accumulators.  The first attempt parks the thread in hardware for a bounded
// time and nearly always succeeds; the timed loop is kept out of line so that the pass body stays small.
__device__ __noinline__ bool wait_full_slow(Waiter w, uint32_t bar, uint32_t parity) { return w.barrier(bar, parity, ERR_WAIT_FULL); }

__device__ __forceinline__ bool wait_full(Waiter w, uint32_t bar, uint32_t parity)
{
    bool ok = mbar_try(bar, parity);
    if (!ok) ok = wait_full_slow(w, bar, parity);
    return __all_sync(0xffffffffu, ok);
}

// After a pass: the stores become visible to the tensor cores' reads, the tensor-memory accesses are ordered
// before the arrival, and the warp counts one stored chunk of the unit.
__device__ __forceinline__ void pass_done(const EpiConv &E, const EpiCtx &c, uint32_t unit)
{
    tc_fence_before();
    fence_proxy_async();
    __syncwarp();
    if (c.lane == 0) red_release_add(E.done_addr + 4u * unit, 1u);
}

// The common pass: two output lines, one 16-channel chunk, results stored where the next convolution reads them.
// The accumulator columns are left at zero: stacked chains accumulate from their first K-step on.
template <int kRes>
__device__ __forceinline__ void epi_pass2(const EpiConv &E, const EpiCtx &c, uint4 q0, uint4 q1)
{
    const uint32_t ch = (q0.x >> 12) & 0xFu;
    tc_fence_after();
    int acc0[16], acc1[16];
    tmem_ld16_issue(E.tmem0 + q0.z, acc0);
    tmem_ld16_issue(E.tmem0 + q0.w, acc1);
    uint32_t r0[4] = {0, 0, 0, 0}, r1[4] = {0, 0, 0, 0};
    if (kRes) {
        const uint4 a = ld_shared_v4(E.res_thread + q1.z), b = ld_shared_v4(E.res_thread + q1.w);
        r0[0] = a.x ^ 0x80808080u; r0[1] = a.y ^ 0x80808080u; r0[2] = a.z ^ 0x80808080u; r0[3] = a.w ^ 0x80808080u;
        r1[0] = b.x ^ 0x80808080u; r1[1] = b.y ^ 0x80808080u; r1[2] = b.z ^ 0x80808080u; r1[3] = b.w ^ 0x80808080u;
    }
    tmem_ld_wait();
    tmem_st16_zero(E.tmem0 + q0.z);
    tmem_st16_zero(E.tmem0 + q0.w);
    const uint32_t cbase = E.const_addr + ch * 256u;
    const uint32_t m2 = E.res_m2;
    const long long r2 = E.res_r2;
    uint32_t o0[4], o1[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const ChanConst4 c0 = ld_chan_const_early(cbase + (4 * g + 0) * 16), c1 = ld_chan_const_early(cbase + (4 * g + 1) * 16);
        const ChanConst4 c2 = ld_chan_const_early(cbase + (4 * g + 2) * 16), c3 = ld_chan_const_early(cbase + (4 * g + 3) * 16);
        o0[g] = pack4_sat(requant1<kRes, 0>(acc0[4 * g + 0], c0, r0[g], m2, r2), requant1<kRes, 1>(acc0[4 * g + 1], c1, r0[g], m2, r2),
                          requant1<kRes, 2>(acc0[4 * g + 2], c2, r0[g], m2, r2), requant1<kRes, 3>(acc0[4 * g + 3], c3, r0[g], m2, r2));
        o1[g] = pack4_sat(requant1<kRes, 0>(acc1[4 * g + 0], c0, r1[g], m2, r2), requant1<kRes, 1>(acc1[4 * g + 1], c1, r1[g], m2, r2),
                          requant1<kRes, 2>(acc1[4 * g + 2], c2, r1[g], m2, r2), requant1<kRes, 3>(acc1[4 * g + 3], c3, r1[g], m2, r2));
    }
    const uint4 v0 = make_uint4(o0[0], o0[1], o0[2], o0[3]), v1 = make_uint4(o1[0], o1[1], o1[2], o1[3]);
    const uint32_t a0 = E.out_thread + q1.x, a1 = E.out_thread + q1.y;
    st_shared_v4(a0, v0);
    st_shared_v4(a1, v1);
    if (E.dup_delta) {
        // first row of a lower band: also the row below the band above it; last row of an upper band: the row above
        // the next band
        st_shared_v4_if(a0 + E.dup_delta, v0, (q0.x >> 16) & E.dup_up);
        st_shared_v4_if(a0 - E.dup_delta, v0, (q0.x >> 17) & E.dup_dn);
        st_shared_v4_if(a1 + E.dup_delta, v1, (q0.x >> 18) & E.dup_up);
        st_shared_v4_if(a1 - E.dup_delta, v1, (q0.x >> 19) & E.dup_dn);
    }
}

// The items (unit, chunk) of a convolution that belong to this warp's set: one wait, one or two records of two lines
// each, one arrival.
template <int kRes>
__device__ __forceinline__ void epi_conv_fast(Waiter w, const EpiConv &E_in, const EpiCtx &c_in, uint32_t passes, uint32_t n_items,
                                            uint32_t item_bytes)
{
    const EpiConv E = E_in;
    const EpiCtx c = c_in;
#pragma unroll 1
    for (uint32_t i = (uint32_t)c.set; i < n_items; i += kSets) {
        const uint32_t rec = passes + item_bytes * i;
        const uint4 q0 = ld_shared_v4(rec), q1 = ld_shared_v4(rec + 16u);
        if (!wait_full(w, E.full_addr + 8u * (q0.x & 0xFFu), E.parity)) return;     // aborted: every other wait falls through too
        epi_pass2<kRes>(E, c, q0, q1);
        if (item_bytes > 32u) {
            const uint4 p0 = ld_shared_v4(rec + 32u), p1 = ld_shared_v4(rec + 48u);
            epi_pass2<kRes>(E, c, p0, p1);
        }
        tmem_st_wait();
        pass_done(E, c, q0.x & 0xFFu);
    }
}

// Stride 2: stores one position's 16 channels of a plane where the output's layout wants them (`line` is the ordinal
// of an even input line; even columns and even rows survive), with the copies that the line layout asks for.
__device__ __noinline__ void store_strided(uint32_t desc, uint32_t sbase, uint32_t lane_idx, uint32_t ch, uint32_t line, uint4 o)
{
    const uint4 h6 = ld_shared_v4(desc + offsetof(LConvDesc, out_base));       // out_base, out_plane, out_pitch16, out_n_lines
    const uint4 h7 = ld_shared_v4(desc + offsetof(LConvDesc, out_log_lines));  // out_log_lines, out_nb, out_logI, res_base
    const uint4 h8 = ld_shared_v4(desc + offsetof(LConvDesc, res_plane));      // res_plane, in_logI, in_I, in_n_lines
    const uint32_t x_i = lane_idx >> h8.y, band_i = (lane_idx & (h8.z - 1u)) >> 2, s = lane_idx & 3u;
    const uint32_t r_i = 2u * line + band_i * h8.w;
    if ((x_i & 1u) || (r_i & 1u)) return;
    const uint32_t r_o = r_i >> 1, x_o = x_i >> 1;
    const uint32_t oline = r_o & (h6.w - 1u);
    const uint32_t olane = (x_o << h7.z) + ((r_o >> h7.x) << 2) + s;
    const uint32_t addr = sbase + h6.x + ch * h6.y + (oline * h6.z + olane) * 16u;
    st_shared_v4(addr, o);
    const uint32_t band = (olane >> 2) & (h7.y - 1u);
    // first row of a lower band: also the row below the band above it; last row of an upper band: the row above the next
    if (oline == 0 && band >= 1) st_shared_v4(addr + (h6.w * h6.z - 4u) * 16u, o);
    if (oline == h6.w - 1u && band + 1u < h7.y) st_shared_v4(addr - (h6.w * h6.z - 4u) * 16u, o);
}

// The general pass (strided convolutions, a lower clamp above -128, a lone line): one line at a time, every
// property decided at run time.  The networks of the benchmark reach it in their two strided shortcuts only.
__device__ __noinline__ void epi_conv_general(Waiter w, const EpiConv &E, const EpiCtx &c, uint32_t desc, uint32_t flags, int32_t lo,
                                              uint32_t passes, uint32_t n_passes)
{
    const bool res = flags & CF_RES, scatter = flags & CF_SCATTER;
    for (uint32_t i = (uint32_t)c.set; i < n_passes; i += kSets) {
        const uint4 q0 = ld_shared_v4(passes + 32u * i), q1 = ld_shared_v4(passes + 32u * i + 16u);
        const uint32_t unit = q0.x & 0xFFu, ch = (q0.x >> 12) & 0xFu, n = (q0.x >> 8) & 0xFu;
        if (!wait_full(w, E.full_addr + 8u * unit, E.parity)) return;
        tc_fence_after();
        for (uint32_t j = 0; j < n; ++j) {
            const uint32_t tcol = j ? q0.w : q0.z, out = j ? q1.y : q1.x, rs = j ? q1.w : q1.z;
            int acc[16];
            tmem_ld16(E.tmem0 + tcol, acc);
            tmem_st16_zero(E.tmem0 + tcol);
            uint4 rv = make_uint4(0, 0, 0, 0);
            if (res) rv = ld_shared_v4(E.res_thread + rs);
            const uint32_t rw[4] = {rv.x ^ 0x80808080u, rv.y ^ 0x80808080u, rv.z ^ 0x80808080u, rv.w ^ 0x80808080u};
            uint32_t o[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                int y[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const ChanConst4 cs = ld_chan_const_early(E.const_addr + ch * 256u + (4 * g + k) * 16);
                    const long long prod = mul_wide(acc[4 * g + k] + cs.bias, cs.mult);
                    int v = cs.s ? (hi32(prod) + cs.c) >> cs.s : hi32(prod) + (int)((uint32_t)lo32(prod) >> 31) + cs.c;
                    if (res) v += hi32(mad_wide_u((rw[g] >> (8 * k)) & 0xFFu, E.res_m2, E.res_r2));
                    y[k] = max(v, lo);
                }
                o[g] = pack4_sat(y[0], y[1], y[2], y[3]);
            }
            const uint4 v = make_uint4(o[0], o[1], o[2], o[3]);
            if (scatter) {
                store_strided(desc, c.sbase, c.lane_idx, ch, (q0.y >> (8 * j)) & 0xFFu, v);
            } else {
                const uint32_t addr = E.out_thread + out;
                st_shared_v4(addr, v);
                if (E.dup_delta) {
                    if (((q0.x >> (16 + 2 * j)) & 1u) & E.dup_up) st_shared_v4(addr + E.dup_delta, v);
                    if (((q0.x >> (17 + 2 * j)) & 1u) & E.dup_dn) st_shared_v4(addr - E.dup_delta, v);
                }
            }
        }
        tmem_st_wait();
        pass_done(E, c, unit);
    }
}

__device__ __forceinline__ void epi_conv(const LineParams &p, const EpiCtx &c, uint32_t blob_off, uint32_t cg, int it)
{
    Waiter w{c.ctrl, p.err};
    bool ok = w.barrier(smem_u32(&c.ctrl->wbar[cg % 3]), (cg / 3) & 1, ERR_WAIT_WEIGHTS);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) return;                    // the abort flag is up: every other wait falls through as well
    const uint32_t desc = c.sbase + blob_off;
    const uint4 h0 = ld_shared_v4(desc);
    const uint4 h1 = ld_shared_v4(desc + offsetof(LConvDesc, a_base));
    const uint4 h3 = ld_shared_v4(desc + offsetof(LConvDesc, d_base));
    const uint4 h4 = ld_shared_v4(desc + offsetof(LConvDesc, use_local));
    const uint4 h5 = ld_shared_v4(desc + offsetof(LConvDesc, w_rel));
    const uint4 h6 = ld_shared_v4(desc + offsetof(LConvDesc, out_base));       // out_base, out_plane, out_pitch16, out_n_lines
    const uint4 h7 = ld_shared_v4(desc + offsetof(LConvDesc, out_log_lines));  // out_log_lines, out_nb, out_logI, res_base
    const uint4 h9 = ld_shared_v4(desc + offsetof(LConvDesc, lo));             // lo, res_m2, res_r2
    const uint32_t use = (uint32_t)it * h4.y + h4.x;
    EpiConv E;
    E.tmem0 = c.tmem_lane + ((h1.w > 1 && (use & 1u)) ? h3.y : h3.x);
    E.full_addr = smem_u32(&c.ctrl->bars[h3.z + (use & 1u) * h4.z]);
    E.done_addr = smem_u32(&c.ctrl->stored[h3.w]);
    E.parity = (use >> 1) & 1u;
    E.const_addr = desc + h5.y;
    E.out_thread = c.sbase + h6.x + c.lane_idx * 16u;
    E.res_thread = c.sbase + h7.w + c.lane_idx * 16u;
    const uint32_t band = (c.lane_idx >> 2) & (h7.y - 1u);
    E.dup_delta = h7.y > 1u ? (h6.w * h6.z - 4u) * 16u : 0u;
    E.dup_up = band >= 1u ? 1u : 0u;
    E.dup_dn = band + 1u < h7.y ? 1u : 0u;
    E.res_m2 = h9.y;
    E.res_r2 = (long long)(((unsigned long long)h9.w << 32) | h9.z);
    const uint32_t passes = desc + h5.w, n_passes = h0.y;
    const uint32_t flags = h0.w;
    if (flags & CF_GENERAL) {
        epi_conv_general(w, E, c, desc, flags, (int32_t)h9.x, passes, n_passes);
        return;
    }
    const uint32_t rpi = lds32(desc + offsetof(LConvDesc, recs_per_item));
    if (flags & CF_RSHORT) epi_conv_fast<2>(w, E, c, passes, n_passes / rpi, 32u * rpi);
    else if (flags & CF_RES) epi_conv_fast<1>(w, E, c, passes, n_passes / rpi, 32u * rpi);
    else epi_conv_fast<0>(w, E, c, passes, n_passes / rpi, 32u * rpi);
}

// FILL: the region takes its halo value everywhere
__device__ void fill_phase(const EpiCtx &c, uint32_t off, uint32_t bytes, uint32_t halo)
{
    const uint32_t word = (halo & 0xFFu) * 0x01010101u;
    const uint4 v = make_uint4(word, word, word, word);
    for (uint32_t o = (uint32_t)c.tid * 16u; o < bytes; o += kThreads * 16u) st_shared_v4(c.sbase + off + o, v);
}

// INPUT: one thread = four horizontally adjacent pixels of one sample, all input channels (Def. 3.3, Def. 3.4).
__device__ void input_phase(const LineParams &p, const EpiCtx &c, int grp)
{
    const int H = p.in_H, W = p.in_W, in_c = p.in_c;
    const int wq = W >> 2;
    const int quads = kG * H * wq;
    const uint32_t *__restrict__ cum = p.ns.cum;
    const uint32_t *__restrict__ guide = p.ns.guide;
    const int T = p.ns.T;
    const uint32_t key0 = p.ns.key0, key1 = p.ns.key1, ctr2 = p.ns.ctr2;
    const uint8_t *__restrict__ x = p.x;
    for (int qi = c.tid; qi < quads; qi += kThreads) {
        // consecutive threads take consecutive samples: their stores fall into one 64-byte run
        const int s = qi & (kG - 1);
        const int rem = qi >> 2;
        const int y = rem / wq, x4 = rem - y * wq;
        const long long j = p.ns.first_sample + (long long)grp * kG + s;
        const uint32_t ctr3 = p.ns.ctr3_fixed | (uint32_t)(((j >> 32) & 0xFF) << 8);
        uint32_t px[4] = {0, 0, 0, 0};
        for (int ch = 0; ch < in_c; ++ch) {
            const uint32_t e = (uint32_t)((ch * H + y) * W + 4 * x4);
            const uint4 r = philox4x32_10(make_uint4(e >> 2, (uint32_t)(j & 0xFFFFFFFFll), ctr2, ctr3), key0, key1);
            const uint32_t u[4] = {r.x, r.y, r.z, r.w};
            const uint32_t clean = __ldg(reinterpret_cast<const uint32_t *>(x + e));
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                int v = (int)((clean >> (8 * k)) & 0xFF) + (guide ? noise_level_guided(u[k], cum, guide, T) : noise_level(u[k], cum, T));
                v = min(255, max(0, v));
                px[k] |= (uint32_t)v << (8 * ch);
            }
        }
        // the input has one row band: line = row, position = column * 4 + sample
        const uint32_t pos = (uint32_t)y * p.input_pitch16 + (uint32_t)(4 * x4) * kG + (uint32_t)s;
#pragma unroll
        for (int k = 0; k < 4; ++k) st_shared_v4(c.sbase + p.input_base + (pos + (uint32_t)k * kG) * 16u, make_uint4(px[k], 0, 0, 0));
    }
}

// TAIL, first half: global average pool.  One thread sums one (sample, channel) pair over the pixels and
// requantises it; consecutive threads take the four samples of consecutive channels (one shared-memory wavefront).
__device__ void tail_pool(const LineParams &p, const EpiCtx &c)
{
    const int tail_W = p.tail_W, n_lines = p.tail_n_lines, hw = p.tail_H * p.tail_W;
    for (int q = c.tid; q < kG * p.tail_C; q += kThreads) {
        const int s = q & (kG - 1), ch = q >> 2;
        const uint32_t base = c.sbase + p.tail_base + (uint32_t)(ch >> 4) * p.tail_plane + (uint32_t)(ch & 15);
        int sum = 0;
        for (int i = 0; i < hw; ++i) {
            const int y = i / tail_W, x = i - y * tail_W;
            const int line = y % n_lines, band = y / n_lines;
            const uint32_t pos = (uint32_t)line * p.tail_pitch16 + ((uint32_t)x << p.tail_logI) + (uint32_t)(band * 4 + s);
            int v;
            asm volatile("ld.shared.s8 %0, [%1];" : "=r"(v) : "r"(base + pos * 16u));
            sum += v - p.pool_zp_in;
        }
        long long v = ((long long)sum * p.pool_mult + (1ll << (p.pool_n - 1))) >> p.pool_n;
        v += p.pool_zp_out;
        v = v < p.pool_lo ? p.pool_lo : v;
        v = v > 127 ? 127 : v;
        c.ctrl->pooled[s][ch] = (int32_t)v;
    }
}

// TAIL, second half: FC, argmax and vote; one warp carries one sample (Algorithm 1 steps 1-4).
__device__ void tail_sample(const LineParams &p, const EpiCtx &c, int s, int grp)
{
    const int tail_C = p.tail_C;
    const int n_classes = p.n_classes;
    const long long sample = (long long)grp * kG + s;          // index within this launch
    const bool counted = sample < p.n_samples;
    int best_v = -1000, best_o = 0x7fffffff;
    for (int o0 = 0; o0 < n_classes; o0 += 32) {
        const int o = o0 + c.lane;
        const bool live = o < n_classes;
        const FcConst k = p.fc_c[live ? o : 0];
        const int8_t *wrow = p.fc_w + (size_t)(live ? o : 0) * 64;
        int acc = k.bias;
        for (int cc = 0; cc < tail_C; ++cc) acc += c.ctrl->pooled[s][cc] * (int)__ldg(wrow + cc);
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

__global__ void __launch_bounds__(kThreads, 1) k_line(const __grid_constant__ LineParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem);
    const uint32_t sbase = smem_u32(smem);
    const int warp = (int)warp_uniform(threadIdx.x >> 5), lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < p.n_bars; i += blockDim.x) mbar_init(smem_u32(&ctrl->bars[i]), p.bar_counts[i]);
    if (threadIdx.x == 0) {
        for (int s = 0; s < 3; ++s) mbar_init(smem_u32(&ctrl->wbar[s]), 1);
        mbar_init(smem_u32(&ctrl->drain), kIssuers);
        ctrl->abort_flag = 0;
    }
    for (int i = threadIdx.x; i < 128; i += blockDim.x) ctrl->hist[i] = 0;
    for (int i = threadIdx.x; i < p.n_phases; i += blockDim.x) ctrl->ptab[i] = p.ptab[i];
    for (int i = threadIdx.x; i < p.n_conv; i += blockDim.x) ctrl->csrc[i] = p.conv_src[i];
    for (int i = threadIdx.x; i < kMaxBars; i += blockDim.x) ctrl->stored[i] = 0;
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctrl->tmem_base;

    EpiCtx c;
    c.ctrl = ctrl; c.sbase = sbase;
    c.warp = warp; c.set = warp >> 2; c.quarter = warp & 3; c.lane = lane; c.tid = threadIdx.x;
    c.lane_idx = (uint32_t)((warp & 3) * 32 + lane);
    c.tmem_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const bool issuer = warp >= kEpiWarps && warp < kEpiWarps + kIssuers, loader = warp == kLoaderWarp, epi = warp < kEpiWarps;
    // accumulators of stacked convolutions start from zero
    if (epi) {
        for (uint32_t col = (uint32_t)c.set * 16u; col < (uint32_t)kTmemCols; col += kSets * 16u) tmem_st16_zero(c.tmem_lane + col);
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t ptab = smem_u32(ctrl->ptab);
    const int n_phases = p.n_phases, stop_phase = p.stop_phase;
    bool role_ok = true;
    int it = 0;
    // thread 0 keeps the time the CTA spends in its CTA-wide phases (they run between barriers, so one thread's clock
    // measures them); what is left of the kernel's duration is the convolutions
    if (threadIdx.x == 0) {
        ctrl->cyc[PH_FILL] = ctrl->cyc[PH_INPUT] = ctrl->cyc[PH_TAIL] = 0;
        ctrl->cyc[PH_CONV] = clock64();         // until the end: the start time
    }
    for (int grp = blockIdx.x; grp < p.n_groups; grp += gridDim.x, ++it) {
        PrevConv prev{0u, 0u, 0u};
        int conv_index = 0;
        bool first_phase = true;
        for (int ph = 0; ph < n_phases && ph <= stop_phase; ++ph) {
            const uint4 e = ld_shared_v4(ptab + 16 * ph);
            if (e.x == PH_CONV) {
                const uint32_t cg = (uint32_t)it * (uint32_t)p.n_conv + (uint32_t)conv_index;
                if (issuer) {
                    if (lane == 0 && role_ok && !ctrl->abort_flag)
                        role_ok = issuer_conv(p, ctrl, sbase, tmem, e.y, cg, warp - kEpiWarps, it, prev);
                    __syncwarp();
                } else if (loader) {
                    if (lane == 0 && role_ok && !ctrl->abort_flag && conv_index + 1 < p.n_conv)
                        role_ok = loader_copy(p, ctrl, sbase, conv_index + 1, cg + 1u, it);
                    __syncwarp();
                } else if (!ctrl->abort_flag) {
                    epi_conv(p, c, e.y, cg, it);
                }
                conv_index += 1;
                first_phase = false;
                continue;
            }
            // CTA-wide phase: everything before it is complete in all warps
            tc_fence_before();
            __syncthreads();
            tc_fence_after();
            prev.n_lines = 0;
            if (first_phase) {
                // the first blob of the group: everything of the previous group is complete
                if (loader && lane == 0 && p.n_conv > 0 && role_ok && !ctrl->abort_flag)
                    role_ok = loader_copy(p, ctrl, sbase, 0, (uint32_t)it * (uint32_t)p.n_conv, it);
                first_phase = false;
            }
            // every warp of the CTA takes part in these phases; nothing inside them can raise the abort flag
            const bool live = !ctrl->abort_flag;
            if (threadIdx.x == 0) ctrl->cyc_mark = clock64();
            if (live) {
                if (e.x == PH_FILL) fill_phase(c, e.y, e.z, e.w);
                else if (e.x == PH_INPUT) input_phase(p, c, grp);
                else tail_pool(p, c);
            }
            if (e.x == PH_TAIL) {
                __syncthreads();
                if (live && warp < kG) tail_sample(p, c, warp, grp);
            }
            fence_proxy_async();
            __syncthreads();
            if (threadIdx.x == 0) ctrl->cyc[e.x & 3u] += clock64() - ctrl->cyc_mark;
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    if (threadIdx.x == 0 && p.phase_cycles) {
        const long long total = clock64() - ctrl->cyc[PH_CONV];
        atomicAdd(p.phase_cycles + PH_FILL, (unsigned long long)ctrl->cyc[PH_FILL]);
        atomicAdd(p.phase_cycles + PH_INPUT, (unsigned long long)ctrl->cyc[PH_INPUT]);
        atomicAdd(p.phase_cycles + PH_TAIL, (unsigned long long)ctrl->cyc[PH_TAIL]);
        atomicAdd(p.phase_cycles + PH_CONV, (unsigned long long)(total - ctrl->cyc[PH_FILL] - ctrl->cyc[PH_INPUT] - ctrl->cyc[PH_TAIL]));
    }
    if (!ctrl->abort_flag)
        for (int i = threadIdx.x; i < p.n_classes; i += blockDim.x)
            if (ctrl->hist[i]) atomicAdd(p.counts + i, ctrl->hist[i]);
    if (p.dump)
        for (uint32_t o = threadIdx.x * 16u; o < p.dump_bytes; o += blockDim.x * 16u)
            *reinterpret_cast<uint4 *>(p.dump + o) = ld_shared_v4(sbase + p.dump_off + o);
    // no tensor-core work may be in flight when tensor memory is released
    if (issuer && lane == 0) {
        Waiter w{ctrl, p.err};
        commit_to(smem_u32(&ctrl->drain));
        w.barrier(smem_u32(&ctrl->drain), 0, ERR_WAIT_DRAIN);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// The engine's wait code on a barrier and a counter that nothing ever completes: one CTA, one thread, the limit given by
// the caller.  The first wait must run out and raise the abort flag and the error word; the second must then fall
// through at once.  out[0..1] = what the two waits returned, out[2] = the abort flag, out[3] = nanoseconds spent.
__global__ void k_wait_probe(int32_t *err, unsigned long long limit_ns, int32_t *out)
{
    extern __shared__ __align__(128) uint8_t smem[];
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem);
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&ctrl->bars[0]), 1);
        ctrl->abort_flag = 0;
        ctrl->stored[0] = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) {
        Waiter w{ctrl, err, limit_ns};
        const unsigned long long t0 = globaltimer();
        out[0] = w.barrier(smem_u32(&ctrl->bars[0]), 0, ERR_WAIT_FULL) ? 1 : 0;
        out[1] = w.counter(smem_u32(&ctrl->stored[0]), 1u, ERR_WAIT_DONE) ? 1 : 0;
        out[2] = ctrl->abort_flag;
        out[3] = (int32_t)min(globaltimer() - t0, 0x7FFFFFFFull);
    }
}

// =============================================================================== host planner

int ilog2(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

// Geometry of one tensor in the line layout.
struct LGeo {
    int C = 0, H = 0, W = 0, planes = 0, halo = 0;
    int I = 0, nb = 0, n_lines = 0, pitch = 0;       // positions per column, row bands, lines, line pitch in positions
    uint32_t plane_bytes = 0, bytes = 0, line0 = 0;  // line0: byte offset of line 0, lane 0 within a plane
    int buffer = -1, producer_phase = -1, producer_conv = -1;
    bool scatter_produced = false;
    int last_use_layer = -1;
    bool last_use_as_input = false;
};

bool set_geometry(LGeo &t)
{
    if (t.W != 32 && t.W != 16 && t.W != 8) return false;
    if (t.H != t.W) return false;
    t.planes = (t.C + 15) / 16;
    t.I = 128 / t.W;
    t.nb = t.I / kG;
    t.n_lines = t.H / t.nb;
    t.pitch = 128 + t.I;
    const int positions = t.I + (t.n_lines + 2) * t.pitch + 8;      // leading gap, lines -1 .. n_lines with their gaps, slack
    t.plane_bytes = (uint32_t)positions * 16u;
    t.bytes = t.plane_bytes * (uint32_t)t.planes;
    t.line0 = (uint32_t)(t.I + t.pitch) * 16u;
    return true;
}

struct PlanBuffer { uint32_t bytes = 0, off = 0; int birth = 0, death = 0, halo = 0; };
struct AllocReq { uint32_t bytes; int birth, death, slack; uint32_t *off; int conv; };

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

// A plan that does not fit is not an error (another engine runs the model); the rule that refused it is kept for
// line_plan_probe, and ISC_PLAN_DEBUG=1 prints it.
thread_local int g_plan_rule = 0;
#define PLAN_FAIL(id) do { g_plan_rule = (id); if (getenv("ISC_PLAN_DEBUG")) fprintf(stderr, "line engine: plan rule %d failed\n", id); return false; } while (0)

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

}  // namespace

struct LinePlan {
    int in_c = 0, in_h = 0, in_w = 0, n_classes = 0, n_phases = 0, n_conv = 0, n_bars = 0;
    uint32_t smem_bytes = 0;
    LineParams base;
    std::vector<int> phase_kind;
    std::vector<LGeo> tensors;
    std::vector<uint32_t> tensor_off;
    PhaseEntry *d_ptab = nullptr;
    ConvSrc *d_conv_src = nullptr;
    uint8_t *d_bar_counts = nullptr;
    uint8_t *d_blob = nullptr;
    int8_t *d_fc_w = nullptr;
    FcConst *d_fc_c = nullptr;
    int32_t *d_err = nullptr;
    unsigned long long *d_phase_cycles = nullptr;
    uint8_t *d_dump = nullptr;
    int sm_count = 0;
    bool attr_set = false;
};

namespace {

// What the planner knows about a convolution phase while it builds the operation and pass tables.
struct ConvPlan {
    int layer = -1, phase = -1;
    int in_tensor = -1, out_tensor = -1;
    bool stacked = false, scatter = false, general = false;
    int recs_per_item = 1;              // records of the pass table per (unit, chunk)
    int m = 0;                          // output lines (ordinals)
    int n_chunks = 0, cols = 0, n_banks = 1;
    int cls = -1, use_local = 0;
    std::vector<LOp> ops;
    std::vector<LPass> passes;
    std::vector<int> done_time;         // per output line: index of the pass that stores its last chunk
    int n_units = 0;
    std::vector<int> unit_of;           // per output line: its unit
    std::vector<int> a_delta;
    std::vector<uint32_t> a_lbo;
    std::vector<std::pair<int, int>> kunits;   // per K-step: indices into `units` (second may be -1)
    struct Unit { int r, s, pl; };             // vertical tap (-1 when stacked), horizontal tap, input plane
    std::vector<Unit> units;
};

bool build_plan(const LayerIn *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes, LinePlan *plan,
                std::vector<uint8_t> *blob_out, std::vector<uint32_t> *blob_offsets, std::vector<PhaseEntry> *ptab_out,
                std::vector<ConvSrc> *csrc_out, std::vector<uint8_t> *bar_counts_out)
{
    const int n_conv_layers = n_layers - 2;
    // ---- tensors of the model (tensor t = output of layer t-1)
    std::vector<LGeo> T((size_t)n_layers + 1);
    T[0].C = in_c; T[0].H = in_h; T[0].W = in_w; T[0].halo = layers[0].d.zp_in;
    for (int i = 0; i < n_conv_layers; ++i) {
        const isc_layer &L = layers[i].d;
        const LGeo &in = T[(size_t)L.in_tensor];
        LGeo &o = T[(size_t)i + 1];
        o.C = L.cout;
        o.H = (in.H + 2 * L.pad - L.kh) / L.stride + 1;
        o.W = (in.W + 2 * L.pad - L.kw) / L.stride + 1;
        o.halo = L.zp_out;
        if (L.stride == 2 && ((in.H & 1) || (in.W & 1))) PLAN_FAIL(1);
    }
    for (int t = 0; t <= n_conv_layers; ++t)
        if (!set_geometry(T[(size_t)t])) PLAN_FAIL(2);
    if (T[0].nb != 1) PLAN_FAIL(3);                 // the input writer knows one row band only
    for (int i = 0; i < n_layers; ++i) {
        const isc_layer &L = layers[i].d;
        T[(size_t)L.in_tensor].last_use_layer = i;
        T[(size_t)L.in_tensor].last_use_as_input = true;
        if (L.res_tensor >= 0) {
            T[(size_t)L.res_tensor].last_use_layer = i;
            T[(size_t)L.res_tensor].last_use_as_input = false;
        }
    }
    // ---- phase skeleton: FILL(input) INPUT, then per convolution [FILL of a fresh output] CONV, then TAIL
    struct Skel { int kind; int layer; int tensor; };
    std::vector<Skel> skel;
    std::vector<PlanBuffer> buffers;
    std::vector<int> layer_phase((size_t)n_layers, -1);
    auto new_buffer = [&](int tensor) {
        PlanBuffer b;
        b.bytes = T[(size_t)tensor].bytes; b.halo = T[(size_t)tensor].halo;
        b.birth = (int)skel.size();
        buffers.push_back(b);
        T[(size_t)tensor].buffer = (int)buffers.size() - 1;
        skel.push_back({PH_FILL, -1, tensor});
    };
    new_buffer(0);
    skel.push_back({PH_INPUT, -1, 0});
    int prev_conv_layer = -1;
    for (int i = 0; i < n_conv_layers; ++i) {
        const isc_layer &L = layers[i].d;
        const int out_t = i + 1;
        LGeo &o = T[(size_t)out_t];
        bool placed = false;
        // (a) in place over the residual operand, when this layer is its last reader
        if (L.res_tensor >= 0 && L.stride == 1 && T[(size_t)L.res_tensor].last_use_layer == i &&
            L.res_tensor != L.in_tensor && T[(size_t)L.res_tensor].halo == o.halo &&
            T[(size_t)L.res_tensor].bytes == o.bytes && T[(size_t)L.res_tensor].W == o.W) {
            o.buffer = T[(size_t)L.res_tensor].buffer;
            placed = true;
        }
        // (b) over a same-shaped tensor whose last reader was the previous convolution, as its input
        if (!placed && L.stride == 1 && prev_conv_layer >= 0)
            for (int t = 1; t <= n_conv_layers && !placed; ++t) {
                const LGeo &x = T[(size_t)t];
                if (x.buffer < 0 || t == out_t || t == L.in_tensor || t == L.res_tensor) continue;
                if (x.last_use_layer != prev_conv_layer || !x.last_use_as_input) continue;
                if (x.C != o.C || x.H != o.H || x.W != o.W || x.halo != o.halo) continue;
                bool newest = true;           // x must be the current tenant of its buffer
                for (int u = t + 1; u <= n_conv_layers; ++u)
                    if (T[(size_t)u].buffer == x.buffer) newest = false;
                if (newest) { o.buffer = x.buffer; placed = true; }
            }
        if (!placed) new_buffer(out_t);
        layer_phase[(size_t)i] = (int)skel.size();
        skel.push_back({PH_CONV, i, -1});
        prev_conv_layer = i;
    }
    const int tail_phase = (int)skel.size();
    skel.push_back({PH_TAIL, -1, n_conv_layers});
    layer_phase[(size_t)n_layers - 2] = tail_phase;
    layer_phase[(size_t)n_layers - 1] = tail_phase;
    const int n_phases = (int)skel.size();
    if (n_phases > kMaxPhases) PLAN_FAIL(4);
    // ---- lifetimes
    for (int t = 0; t <= n_conv_layers; ++t) {
        LGeo &x = T[(size_t)t];
        if (x.buffer < 0) PLAN_FAIL(5);
        int death = x.last_use_layer >= 0 ? layer_phase[(size_t)x.last_use_layer] : -1;
        x.producer_phase = t >= 1 ? layer_phase[(size_t)t - 1] : 1;
        death = std::max(death, x.producer_phase);
        buffers[(size_t)x.buffer].death = std::max(buffers[(size_t)x.buffer].death, death);
    }
    // ---- convolutions: K-steps, operations, passes
    std::vector<ConvPlan> convs;
    std::map<std::pair<int, int>, int> class_of;            // (lines, chunks) -> class
    std::vector<int> class_lines, class_chunks, class_uses;
    for (int ph = 0; ph < n_phases; ++ph) {
        if (skel[(size_t)ph].kind != PH_CONV) continue;
        ConvPlan cp;
        cp.layer = skel[(size_t)ph].layer; cp.phase = ph;
        const isc_layer &L = layers[cp.layer].d;
        cp.in_tensor = L.in_tensor; cp.out_tensor = cp.layer + 1;
        LGeo &in = T[(size_t)cp.in_tensor];
        LGeo &out = T[(size_t)cp.out_tensor];
        out.producer_conv = (int)convs.size();
        cp.scatter = L.stride == 2;
        out.scatter_produced = cp.scatter;
        cp.n_chunks = L.cout / 16; cp.cols = L.cout;
        if (cp.scatter && (in.n_lines & 1)) PLAN_FAIL(6);
        cp.m = cp.scatter ? in.n_lines / 2 : in.n_lines;
        if (cp.m > kMaxLines || cp.m * cp.cols > kTmemCols) PLAN_FAIL(7);
        cp.stacked = L.kh == 3 && L.stride == 1 && 3 * L.cout <= 128 && in.n_lines >= 2;
        cp.n_banks = kTmemCols / (cp.m * cp.cols) >= 2 ? 2 : 1;
        if (L.res_tensor >= 0) {
            const LGeo &r = T[(size_t)L.res_tensor];
            if (cp.scatter || r.W != out.W || r.H != out.H || r.C != out.C) PLAN_FAIL(8);
            const int res_n = 31 - L.res_shift;
            if (res_n != 31 && res_n != 32) PLAN_FAIL(9);
        }
        // K units and steps
        const int s_lo = L.kw == 3 ? -1 : 0, s_hi = L.kw == 3 ? 1 : 0;
        if (cp.stacked) {
            for (int pl = 0; pl < in.planes; ++pl)
                for (int s = s_lo; s <= s_hi; ++s) cp.units.push_back({-1, s, pl});
        } else {
            const int r_lo = L.kh == 3 ? 0 : 1, r_hi = L.kh == 3 ? 2 : 1;
            for (int pl = 0; pl < in.planes; ++pl)
                for (int r = r_lo; r <= r_hi; ++r)
                    for (int s = s_lo; s <= s_hi; ++s) cp.units.push_back({r, s, pl});
        }
        auto unit_addr = [&](const ConvPlan::Unit &u) {
            const int dr = cp.stacked ? 0 : u.r - 1;
            return (long long)u.pl * in.plane_bytes + ((long long)dr * in.pitch + (long long)u.s * in.I) * 16;
        };
        for (size_t a = 0; a < cp.units.size(); a += 2) {
            if (a + 1 < cp.units.size()) {
                const long long d = unit_addr(cp.units[a + 1]) - unit_addr(cp.units[a]);
                if (d <= 0 || d >= (1 << 18)) PLAN_FAIL(10);
                cp.kunits.push_back({(int)a, (int)a + 1});
                cp.a_delta.push_back((int)unit_addr(cp.units[a]));
                cp.a_lbo.push_back((uint32_t)d);
            } else {
                cp.kunits.push_back({(int)a, -1});
                cp.a_delta.push_back((int)unit_addr(cp.units[a]));
                cp.a_lbo.push_back(16u);
            }
        }
        if ((int)cp.kunits.size() > kMaxKsteps) PLAN_FAIL(11);
        // ---- operations
        const ConvPlan *pv = (!convs.empty() && convs.back().phase == ph - 1) ? &convs.back() : nullptr;
        // same lines and chunks: the same barriers (class) and, with one bank, the same accumulator columns
        const bool same_class = pv && pv->m == cp.m && pv->n_chunks == cp.n_chunks;
        // the previous convolution produced this one's input, line for line
        const bool aligned = pv && in.producer_conv == (int)convs.size() - 1 && !pv->scatter;
        // Same class: the same barriers, and with one bank the same accumulator columns.  An operation then waits for
        // the previous convolution's lines of the same numbers as the output lines it adds to, so that no line of
        // this convolution can be stored (and arrive on the line's barrier) before that line of the previous one.
        const bool slots = same_class;
        auto prev_time = [&](int line) { return pv ? pv->done_time[(size_t)line] : 0; };
        auto src_line = [&](int p) -> int {       // which output line of the producer fills input line p (-1: constant)
            if (p >= 0 && p < in.n_lines) return p;
            if (in.nb == 1) return -1;
            return p < 0 ? in.n_lines - 1 : 0;
        };
        struct ProtoOp { int a_line, b_block, n_blocks, d_line; std::vector<int> need; std::vector<int> outs; int ready; };
        std::vector<ProtoOp> proto;
        if (cp.stacked) {
            for (int p = -1; p <= in.n_lines; ++p) {
                ProtoOp o;
                o.a_line = p;
                const int y_lo = std::max(p - 1, 0), y_hi = std::min(p + 1, in.n_lines - 1);
                o.b_block = y_lo - (p - 1); o.n_blocks = y_hi - y_lo + 1; o.d_line = y_lo;
                for (int y = y_lo; y <= y_hi; ++y) o.outs.push_back(y);
                if (aligned && src_line(p) >= 0) o.need.push_back(src_line(p));
                if (slots) for (int y = y_lo; y <= y_hi; ++y) o.need.push_back(y);
                proto.push_back(o);
            }
        } else {
            for (int j = 0; j < cp.m; ++j) {
                ProtoOp o;
                const int cline = cp.scatter ? 2 * j : j;
                o.a_line = cline; o.b_block = 0; o.n_blocks = 1; o.d_line = j;
                o.outs.push_back(j);
                if (aligned)
                    for (int r = (L.kh == 3 ? -1 : 0); r <= (L.kh == 3 ? 1 : 0); ++r)
                        if (src_line(cline + r) >= 0) o.need.push_back(src_line(cline + r));
                if (slots) o.need.push_back(j);
                proto.push_back(o);
            }
        }
        for (ProtoOp &o : proto) {
            o.ready = 0;
            for (int l : o.need) o.ready = std::max(o.ready, prev_time(l));
        }
        std::stable_sort(proto.begin(), proto.end(), [](const ProtoOp &a, const ProtoOp &b) { return a.ready < b.ready; });
        // completion of each output line = the last operation that contributes to it
        std::vector<int> last_op((size_t)cp.m, -1);
        for (size_t i = 0; i < proto.size(); ++i)
            for (int y : proto[i].outs) last_op[(size_t)y] = (int)i;
        // ---- units: the lines of a pass, in the order of completion; one barrier pair per unit
        std::vector<int> order((size_t)cp.m);
        for (int y = 0; y < cp.m; ++y) order[(size_t)y] = y;
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return last_op[(size_t)a] < last_op[(size_t)b]; });
        // A record of the pass table covers `sup` lines; a unit (one "accumulators complete" barrier, one "stored"
        // counter) covers `upl` lines = one or two records.  Long convolutions take four-line units: every barrier
        // arrival costs an issuing thread a tcgen05.commit and every unit costs an epilogue warp a wait and an arrival.
        const int sup = cp.m >= 2 ? 2 : 1;
        bool general = cp.scatter || (cp.m & 1) || (L.relu && L.zp_out > -128);
        for (int oc = 0; oc < L.cout; ++oc) general = general || layers[cp.layer].shift[oc] == 1;
        cp.general = general;
        const int upl = (!general && cp.m >= 16 && cp.m % 4 == 0) ? 4 : sup;
        cp.recs_per_item = upl / sup;
        cp.n_units = (cp.m + upl - 1) / upl;
        cp.unit_of.assign((size_t)cp.m, 0);
        std::vector<int> unit_last_op((size_t)cp.n_units, -1);
        for (int i = 0; i < cp.m; ++i) {
            const int u = i / upl;
            cp.unit_of[(size_t)order[(size_t)i]] = u;
            unit_last_op[(size_t)u] = std::max(unit_last_op[(size_t)u], last_op[(size_t)order[(size_t)i]]);
        }
        // class: same number of units and chunks = same barriers
        const auto key = std::make_pair(cp.n_units, cp.n_chunks);
        if (!class_of.count(key)) {
            class_of[key] = (int)class_lines.size();
            class_lines.push_back(cp.n_units); class_chunks.push_back(cp.n_chunks); class_uses.push_back(0);
        }
        cp.cls = class_of[key];
        cp.use_local = class_uses[(size_t)cp.cls]++;
        const bool wait_all = pv && pv->cls != cp.cls;
        // Record i belongs to issuing thread i mod kIssuers; every thread needs a record to carry its arrivals.
        auto null_op = []() { ProtoOp o; o.a_line = 0; o.b_block = 0; o.n_blocks = 0; o.d_line = 0; o.ready = 0; return o; };
        while (proto.size() < (size_t)kIssuers) proto.push_back(null_op());
        // Each thread arrives on every unit's barrier once: after its last record that adds to the unit, or with any
        // of its records if it has none (at most three arrivals fit a record; empty records are added as needed).
        std::vector<std::vector<int>> commits;
        for (int attempt = 0;; ++attempt) {
            commits.assign(proto.size(), std::vector<int>());
            bool fits = true;
            std::vector<std::vector<char>> has((size_t)cp.n_units, std::vector<char>((size_t)kIssuers, 0));
            for (int u = 0; u < cp.n_units && fits; ++u)
                for (int wi = 0; wi < kIssuers && fits; ++wi) {
                    int last = -1;
                    for (size_t i = (size_t)wi; i < proto.size(); i += kIssuers)
                        for (int y : proto[i].outs)
                            if (cp.unit_of[(size_t)y] == u) last = (int)i;
                    if (last < 0) continue;
                    if (commits[(size_t)last].size() >= 3) fits = false;
                    else { commits[(size_t)last].push_back(u); has[(size_t)u][(size_t)wi] = 1; }
                }
            for (int u = 0; u < cp.n_units && fits; ++u)
                for (int wi = 0; wi < kIssuers && fits; ++wi) {
                    if (has[(size_t)u][(size_t)wi]) continue;
                    int carrier = -1;
                    for (size_t i = (size_t)wi; i < proto.size() && carrier < 0; i += kIssuers)
                        if (commits[i].size() < 3) carrier = (int)i;
                    if (carrier < 0) fits = false;
                    else commits[(size_t)carrier].push_back(u);
                }
            if (fits) break;
            if (attempt >= 8) PLAN_FAIL(13);
            while (proto.size() % kIssuers) proto.push_back(null_op());
            for (int wi = 0; wi < kIssuers; ++wi) proto.push_back(null_op());
        }
        // No thread may still be reading the table when the convolution is complete (its blob's place may then be
        // reused): every thread's last record must carry an arrival, so empty records at the end are dropped.
        while (!proto.empty() && proto.back().n_blocks == 0 && commits.back().empty()) { proto.pop_back(); commits.pop_back(); }
        for (int wi = 0; wi < kIssuers; ++wi) {
            int last = -1;
            for (size_t i = (size_t)wi; i < proto.size(); i += kIssuers) last = (int)i;
            if (last < 0 || commits[(size_t)last].empty()) PLAN_FAIL(23);
        }
        // each thread waits, once, for what its own records need
        std::vector<std::vector<char>> waited((size_t)kIssuers, std::vector<char>(pv ? (size_t)pv->n_units : 0, 0));
        std::vector<char> all_waited(pv ? (size_t)pv->n_units : 0, 0);
        for (size_t i = 0; i < proto.size(); ++i) {
            const ProtoOp &o = proto[i];
            const size_t wi = i % kIssuers;
            LOp op;
            memset(&op, 0xFF, sizeof(op));
            op.flags = o.n_blocks == 0 ? OPF_NULL : 0;
            op.d_col = (uint32_t)(o.d_line * cp.cols);
            const uint32_t a_fmt_bit = cp.in_tensor == 0 ? 0u : 1u;
            op.idesc = (2u << 4) | (a_fmt_bit << 7) | (1u << 10) | ((uint32_t)((std::max(o.n_blocks, 1) * L.cout) >> 3) << 17) | ((128u >> 4) << 24);
            op.a_add = (uint32_t)(o.a_line + 1) * (uint32_t)in.pitch;
            op.b_add = (uint32_t)o.b_block * (uint32_t)L.cout * 2u;
            if (i < (size_t)kIssuers && wait_all) {
                op.flags |= OPF_WAIT_ALL;
                std::fill(waited[wi].begin(), waited[wi].end(), 1);
            }
            int n_wait = 0, n_commit = 0;
            std::vector<int> need_units;
            for (int l : o.need) need_units.push_back(pv->unit_of[(size_t)l]);
            // A thread may arrive on a unit's barrier only when the barrier's previous use is over.  Between
            // convolutions of one class that use is the previous convolution's unit of the same number; anything
            // older is complete once the previous convolution is (the thread's first record has waited for all of it).
            if (pv && pv->cls == cp.cls)
                for (int u : commits[i]) need_units.push_back(u);
            for (int u : need_units)
                if (!waited[wi][(size_t)u]) {
                    if (n_wait >= 4) PLAN_FAIL(12);
                    op.wait[n_wait++] = (uint16_t)(4 * u);
                    waited[wi][(size_t)u] = 1;
                    all_waited[(size_t)u] = 1;
                }
            for (int u : commits[i]) op.commit[n_commit++] = (uint16_t)(8 * u);
            // unused wait slots repeat the first one, so that the kernel reads two (or four) counters without looking
            if (n_wait) {
                op.flags |= OPF_WAITS | (n_wait > 2 ? OPF_WAITS4 : 0);
                for (int k = n_wait; k < 4; ++k) op.wait[k] = op.wait[0];
            }
            op.flags |= (uint16_t)(n_wait << 4) | (uint16_t)(n_commit << 8);
            cp.ops.push_back(op);
        }
        // "this convolution complete" must imply "the previous one complete": between them the threads wait for all its units
        if (pv && !wait_all)
            for (char wtd : all_waited)
                if (!wtd) PLAN_FAIL(20);
        // ---- passes: unit by unit, chunk by chunk
        cp.done_time.assign((size_t)cp.m, 0);
        int n_items = 0;
        for (int u = 0; u < cp.n_units; ++u)
            for (int ch = 0; ch < cp.n_chunks; ++ch, ++n_items)
              for (int rec = 0; rec < cp.recs_per_item; ++rec) {
                const int first = u * upl + rec * sup;
                const int n = std::min(sup, cp.m - first);
                LPass P;
                memset(&P, 0, sizeof(P));
                P.meta = (uint32_t)u | ((uint32_t)n << 8) | ((uint32_t)ch << 12);
                for (int q = 0; q < n; ++q) {
                    const int line = order[(size_t)first + q];
                    P.lines |= (uint32_t)line << (8 * q);
                    P.tcol[q] = (uint32_t)(line * cp.cols + ch * 16);
                    P.out[q] = (uint32_t)(line * out.pitch) * 16u + (uint32_t)ch * out.plane_bytes;
                    P.res[q] = L.res_tensor >= 0 ? (uint32_t)(line * out.pitch) * 16u + (uint32_t)ch * T[(size_t)L.res_tensor].plane_bytes : 0u;
                    if (!cp.scatter) {
                        if (line == 0) P.meta |= 1u << (16 + 2 * q);
                        if (line == out.n_lines - 1) P.meta |= 1u << (17 + 2 * q);
                    }
                    cp.done_time[(size_t)line] = n_items / kSets;
                }
                cp.passes.push_back(P);
              }
        convs.push_back(cp);
    }
    const int n_conv = (int)convs.size();
    if (n_conv > kMaxConv) PLAN_FAIL(22);
    // ---- barriers: per class, one per output line for "accumulators complete" and one for "line stored"
    std::vector<int> class_full(class_lines.size()), class_done(class_lines.size());
    bar_counts_out->clear();
    for (size_t k = 0; k < class_lines.size(); ++k) {
        class_full[k] = (int)bar_counts_out->size();
        for (int l = 0; l < 2 * class_lines[k]; ++l) bar_counts_out->push_back((uint8_t)kIssuers);    // two sets, one arrival per issuing thread
        class_done[k] = (int)bar_counts_out->size();
        for (int l = 0; l < class_lines[k]; ++l) bar_counts_out->push_back((uint8_t)(4 * class_chunks[k]));
    }
    if ((int)bar_counts_out->size() > kMaxBars) PLAN_FAIL(14);
    // ---- blob sizes and shared-memory placement in order of birth
    std::vector<uint32_t> w_bytes((size_t)n_conv), w_off((size_t)n_conv), w_rel((size_t)n_conv), c_rel((size_t)n_conv),
        ops_rel((size_t)n_conv), passes_rel((size_t)n_conv);
    for (int c = 0; c < n_conv; ++c) {
        const ConvPlan &cp = convs[(size_t)c];
        const isc_layer &L = layers[cp.layer].d;
        const uint32_t rows = (uint32_t)(cp.stacked ? 3 : 1) * (uint32_t)L.cout;
        uint32_t at = (uint32_t)sizeof(LConvDesc);
        ops_rel[(size_t)c] = at; at += ((uint32_t)cp.ops.size() + (uint32_t)kIssuers) * (uint32_t)sizeof(LOp);    // spare records: reads run one ahead
        passes_rel[(size_t)c] = at; at += (uint32_t)cp.passes.size() * (uint32_t)sizeof(LPass);
        at = (at + 127u) & ~127u;
        w_rel[(size_t)c] = at; at += (uint32_t)cp.kunits.size() * rows * 32u;
        c_rel[(size_t)c] = at; at += (uint32_t)L.cout * 16u;
        w_bytes[(size_t)c] = (at + 127u) & ~127u;
    }
    std::vector<AllocReq> reqs, placed;
    for (PlanBuffer &b : buffers) reqs.push_back({b.bytes, b.birth, b.death, 0, &b.off, -1});
    for (int c = 0; c < n_conv; ++c)
        reqs.push_back({w_bytes[(size_t)c], c == 0 ? 0 : convs[(size_t)c - 1].phase, convs[(size_t)c].phase, c == 0 ? 0 : 1,
                        &w_off[(size_t)c], c});
    std::stable_sort(reqs.begin(), reqs.end(), [](const AllocReq &a, const AllocReq &b) { return a.birth < b.birth; });
    uint32_t high = kCtrlBytes;
    std::vector<char> late((size_t)n_conv, 0);
    for (AllocReq &r : reqs) {
        bool ok = place(placed, r, kSmemLimit);
        if (!ok && r.conv > 0) {
            // A blob is normally copied when the convolution before its own starts, while the one before that may
            // still be in its epilogue (slack 1).  Where that does not fit, it is copied once that one is complete.
            r.slack = 0;
            late[(size_t)r.conv] = 1;
            ok = place(placed, r, kSmemLimit);
        }
        if (!ok) {
            if (getenv("ISC_PLAN_DEBUG")) {
                fprintf(stderr, "line engine: no room for %u bytes born at phase %d (dies %d); busy then:\n", r.bytes, r.birth, r.death);
                for (const AllocReq &e : placed)
                    if (e.death >= r.birth - r.slack)
                        fprintf(stderr, "  [%u, %u) phases %d..%d\n", *e.off, *e.off + e.bytes, e.birth, e.death);
            }
            PLAN_FAIL(15);
        }
        high = std::max(high, *r.off + r.bytes);
        if (getenv("ISC_PLAN_DEBUG") && atoi(getenv("ISC_PLAN_DEBUG")) > 1)
            fprintf(stderr, "  %s %d: [%u, %u) phases %d..%d\n", r.conv >= 0 ? "blob" : "tensor", r.conv, *r.off, *r.off + r.bytes, r.birth, r.death);
    }
    plan->tensors = T;
    plan->tensor_off.assign(T.size(), 0);
    for (int t = 0; t <= n_conv_layers; ++t) plan->tensor_off[(size_t)t] = buffers[(size_t)T[(size_t)t].buffer].off;
    // ---- emit phases and blobs
    ptab_out->assign((size_t)n_phases, PhaseEntry{0, 0, 0, 0});
    csrc_out->assign((size_t)n_conv, ConvSrc{0, 0, 0, 0, 0, 0, 0});
    blob_out->clear();
    blob_offsets->assign((size_t)n_conv, 0);
    plan->phase_kind.assign((size_t)n_phases, 0);
    int conv_at = 0;
    for (int ph = 0; ph < n_phases; ++ph) {
        const Skel &S = skel[(size_t)ph];
        PhaseEntry &E = (*ptab_out)[(size_t)ph];
        E.kind = (uint32_t)S.kind;
        plan->phase_kind[(size_t)ph] = S.kind;
        if (S.kind == PH_FILL) {
            E.a = plan->tensor_off[(size_t)S.tensor]; E.b = T[(size_t)S.tensor].bytes; E.c = (uint32_t)(T[(size_t)S.tensor].halo & 0xFF);
            continue;
        }
        if (S.kind != PH_CONV) continue;
        const int c = conv_at++;
        const ConvPlan &cp = convs[(size_t)c];
        const LayerIn &ML = layers[cp.layer];
        const isc_layer &L = ML.d;
        const LGeo &in = T[(size_t)cp.in_tensor], &out = T[(size_t)cp.out_tensor];
        E.a = w_off[(size_t)c];
        std::vector<uint8_t> blob(w_bytes[(size_t)c], 0);
        LConvDesc D;
        memset(&D, 0, sizeof(D));
        int32_t res_c = 0;                    // constant of the residual term's short form, folded into the rounding addends
        D.n_ops = (uint32_t)cp.ops.size(); D.n_passes = (uint32_t)cp.passes.size(); D.n_ksteps = (uint32_t)cp.kunits.size();
        D.flags = (cp.stacked ? CF_STACKED : 0u) | (L.res_tensor >= 0 ? CF_RES : 0u) | (cp.scatter ? CF_SCATTER : 0u);
        const int lo = L.relu ? std::max(-128, L.zp_out) : -128;
        if (lo > -128) D.flags |= CF_LO;
        D.lo = lo;
        // the fast pass covers pairs of lines stored in place with the saturating pack as the only clamp
        if (cp.general) D.flags |= CF_GENERAL;
        D.recs_per_item = (uint32_t)cp.recs_per_item;
        // operand base: line -1, lane 0, plane 0 of the input
        D.a_base = plan->tensor_off[(size_t)cp.in_tensor] + in.line0 - (uint32_t)in.pitch * 16u;
        D.pitch16 = (uint32_t)in.pitch;
        D.bblock16 = (uint32_t)L.cout * 2u;
        D.n_banks = (uint32_t)cp.n_banks;
        const uint32_t a_fmt = cp.in_tensor == 0 ? 0u : 1u;
        for (int nbk = 1; nbk <= 3; ++nbk)
            D.idesc[nbk - 1] = (2u << 4) | (a_fmt << 7) | (1u << 10) | ((uint32_t)((nbk * L.cout) >> 3) << 17) | ((128u >> 4) << 24);
        D.cols = (uint32_t)cp.cols;
        D.d_base[0] = 0; D.d_base[1] = cp.n_banks > 1 ? (uint32_t)(cp.m * cp.cols) : 0u;
        D.bar_full = (uint32_t)class_full[(size_t)cp.cls]; D.bar_done = (uint32_t)class_done[(size_t)cp.cls];
        D.use_local = (uint32_t)cp.use_local; D.uses_per_group = (uint32_t)class_uses[(size_t)cp.cls];
        D.n_lines = (uint32_t)cp.n_units; D.n_chunks = (uint32_t)cp.n_chunks;
        D.w_rel = w_rel[(size_t)c]; D.c_rel = c_rel[(size_t)c]; D.ops_rel = ops_rel[(size_t)c]; D.passes_rel = passes_rel[(size_t)c];
        D.out_base = plan->tensor_off[(size_t)cp.out_tensor] + out.line0;
        D.out_plane = out.plane_bytes; D.out_pitch16 = (uint32_t)out.pitch; D.out_n_lines = (uint32_t)out.n_lines;
        D.out_log_lines = (uint32_t)ilog2(out.n_lines); D.out_nb = (uint32_t)out.nb; D.out_logI = (uint32_t)ilog2(out.I);
        if ((1 << D.out_log_lines) != out.n_lines) PLAN_FAIL(16);
        D.in_logI = (uint32_t)ilog2(in.I); D.in_I = (uint32_t)in.I; D.in_n_lines = (uint32_t)in.n_lines;
        if (L.res_tensor >= 0) {
            const LGeo &r = T[(size_t)L.res_tensor];
            D.res_base = plan->tensor_off[(size_t)L.res_tensor] + r.line0;
            D.res_plane = r.plane_bytes;
            const int res_n = 31 - L.res_shift;
            const unsigned long long m2 = (unsigned long long)(uint32_t)L.res_mult << (32 - res_n);
            if (L.res_mult <= 0 || m2 >= (1ull << 32)) PLAN_FAIL(17);
            // rs((r - zp) * mult, n) = floor(((u - 128 - zp) * mult + 2^(n-1)) * 2^(32-n) / 2^32), u = r + 128
            const long long r2 = (((1ll << (res_n - 1)) - (128ll + L.zp_res) * (long long)L.res_mult)) * (1ll << (32 - res_n));
            D.res_m2 = (uint32_t)m2;
            D.res_r2_lo = (uint32_t)((unsigned long long)r2 & 0xFFFFFFFFull);
            D.res_r2_hi = (uint32_t)((unsigned long long)r2 >> 32);
            // the fast pass takes the term without the 64-bit addend when that form exists and its constant fits into
            // every channel's rounding addend
            uint32_t k8 = 0;
            bool short_form = !cp.general && residual_short_form(L.res_mult, L.res_shift, L.zp_res, &k8, &res_c);
            for (int oc = 0; oc < L.cout && short_form; ++oc) {
                const int sft = ML.shift[oc] - 1;
                const long long add = sft >= 1 ? (1ll << (sft - 1)) + ((long long)L.zp_out - res_c) * (1ll << sft) : (1ll << 40);
                short_form = add > -(1ll << 31) && add < (1ll << 31);
            }
            if (short_form) {
                D.flags |= CF_RSHORT;
                D.res_r2_lo = k8;
                D.res_r2_hi = 0;
            } else {
                res_c = 0;
            }
        }
        for (size_t k = 0; k < cp.kunits.size(); ++k) {
            const long long a = (long long)D.a_base + cp.a_delta[k];
            if (a < 0 || (a & 15) || (cp.a_lbo[k] & 15u)) PLAN_FAIL(21);
            D.a_lo[k] = (uint32_t)(a >> 4) | ((cp.a_lbo[k] >> 4) << 16);
        }
        D.b_lo0 = ((w_off[(size_t)c] + w_rel[(size_t)c]) >> 4) | ((128u >> 4) << 16);
        D.kstep16 = (uint32_t)(cp.stacked ? 3 : 1) * (uint32_t)L.cout * 2u;
        // operand reads stay inside the input's region
        for (size_t k = 0; k < cp.kunits.size(); ++k)
            for (const LOp &op : cp.ops) {
                const long long lo_b = (long long)in.line0 - (long long)in.pitch * 16 + (long long)op.a_add * 16 + cp.a_delta[k];
                const long long hi_b = lo_b + cp.a_lbo[k] + 128 * 16;
                if (lo_b < 0 || hi_b > (long long)in.bytes) PLAN_FAIL(18);
            }
        memcpy(blob.data(), &D, sizeof(D));
        memcpy(blob.data() + ops_rel[(size_t)c], cp.ops.data(), cp.ops.size() * sizeof(LOp));
        memcpy(blob.data() + passes_rel[(size_t)c], cp.passes.data(), cp.passes.size() * sizeof(LPass));
        // weights: per K-step, rows = block * cout + oc (block b = vertical tap 2 - b when stacked)
        const int taps = L.kh * L.kw;
        const uint32_t rows = (uint32_t)(cp.stacked ? 3 : 1) * (uint32_t)L.cout;
        for (size_t k = 0; k < cp.kunits.size(); ++k) {
            const int halves[2] = {cp.kunits[k].first, cp.kunits[k].second};
            for (int hf = 0; hf < 2; ++hf) {
                if (halves[hf] < 0) continue;
                const ConvPlan::Unit &u = cp.units[(size_t)halves[hf]];
                for (uint32_t n = 0; n < rows; ++n) {
                    const int oc = (int)(n % (uint32_t)L.cout), blk = (int)(n / (uint32_t)L.cout);
                    const int r = cp.stacked ? 2 - blk : u.r;
                    const int tap = L.kh == 3 ? r * 3 + (u.s + 1) : 0;
                    for (int b = 0; b < 16; ++b) {
                        const int ci = u.pl * 16 + b;
                        if (ci >= L.cin) continue;
                        const int8_t wv = ML.w[((size_t)oc * L.cin + ci) * taps + tap];
                        blob[w_rel[(size_t)c] + k * rows * 32 + (size_t)(n / 8) * 256 + (size_t)hf * 128 + (size_t)(n % 8) * 16 + b] = (uint8_t)wv;
                    }
                }
            }
        }
        bool any_shift_one = false;
        for (int oc = 0; oc < L.cout; ++oc) {
            long long wsum = 0;
            for (int q = 0; q < L.cin * taps; ++q) wsum += ML.w[(size_t)oc * L.cin * taps + q];
            const int sh = ML.shift[oc];
            if (sh < 1 || sh > 20) PLAN_FAIL(19);
            const long long biasf = (long long)ML.bias[oc] - (long long)L.zp_in * wsum;
            if (biasf < -(1ll << 31) || biasf >= (1ll << 31)) PLAN_FAIL(24);
            const int sft = sh - 1;
            const int32_t addend = sft ? (int32_t)((1ll << (sft - 1)) + ((long long)L.zp_out - res_c) * (1ll << sft)) : L.zp_out;
            int32_t cst[4] = {(int32_t)biasf, ML.mult[oc], addend, sft};
            memcpy(&blob[c_rel[(size_t)c] + (size_t)oc * 16], cst, 16);
            if (sft == 0) any_shift_one = true;
        }
        if (any_shift_one && !cp.general) PLAN_FAIL(25);      // a shift of one puts the rounding half in the product's low word
        (*blob_offsets)[(size_t)c] = (uint32_t)blob_out->size();
        blob_out->insert(blob_out->end(), blob.begin(), blob.end());
        (*csrc_out)[(size_t)c].bytes_phase = w_bytes[(size_t)c] | ((uint32_t)ph << 24);
        (*csrc_out)[(size_t)c].smem_off = w_off[(size_t)c] | (late[(size_t)c] ? 0x80000000u : 0u);
        {
            // The copy starts while the convolution before this one runs.  The blob's place was last used by the
            // convolution three back or an earlier one (for a late blob: two back), which must be complete by then.
            const int q = late[(size_t)c] ? c - 2 : c - 3;
            ConvSrc &cs = (*csrc_out)[(size_t)c];
            cs.dep_first = cs.dep_units = cs.dep_mult = cs.dep_local_uses = 0;
            if (q >= 0) {
                const ConvPlan &dq = convs[(size_t)q];
                cs.dep_first = (uint32_t)class_done[(size_t)dq.cls];
                cs.dep_units = (uint32_t)dq.n_units;
                cs.dep_mult = 4u * (uint32_t)dq.n_chunks;
                cs.dep_local_uses = (uint32_t)dq.use_local | ((uint32_t)class_uses[(size_t)dq.cls] << 16);
            }
        }
    }
    plan->n_phases = n_phases;
    plan->n_conv = n_conv;
    plan->n_bars = (int)bar_counts_out->size();
    plan->smem_bytes = (high + 127u) & ~127u;
    (void)n_classes;
    return true;
}

}  // namespace

namespace {

// The structure the engine is built for: convolutions, then global average pool, then FC.
bool structure_ok(const LayerIn *layers, int n_layers, int n_classes)
{
    if (n_layers < 3 || n_classes > 128) PLAN_FAIL(101);
    const isc_layer &LP = layers[n_layers - 2].d, &LF = layers[n_layers - 1].d;
    if (LP.op != ISC_GAVGPOOL || LF.op != ISC_FC) PLAN_FAIL(102);
    if (LP.in_tensor != n_layers - 2 || LF.in_tensor != n_layers - 1) PLAN_FAIL(103);
    if (LP.cin > 64 || LP.cin % 16 != 0 || LF.res_tensor >= 0) PLAN_FAIL(104);
    for (int i = 0; i < n_layers - 2; ++i) {
        const isc_layer &L = layers[i].d;
        if (!conv_ok(L, i == 0)) PLAN_FAIL(105);
        if ((i == 0) != (L.in_tensor == 0)) PLAN_FAIL(106);
        if (L.res_tensor == 0) PLAN_FAIL(107);
        // a consumer's zero-point must be the halo value its operand was written with
        if (L.in_tensor > 0 && L.zp_in != layers[L.in_tensor - 1].d.zp_out) PLAN_FAIL(108);
        if (L.in_tensor > i || L.res_tensor > i) PLAN_FAIL(109);
    }
    if (LP.zp_in != layers[n_layers - 3].d.zp_out) PLAN_FAIL(110);
    return true;
}

}  // namespace

int line_plan_probe(const LayerIn *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes, int *rule, uint32_t *smem_bytes)
{
    g_plan_rule = 0;
    *smem_bytes = 0;
    bool ok = structure_ok(layers, n_layers, n_classes);
    if (ok) {
        LinePlan plan;
        std::vector<uint8_t> blob, bar_counts;
        std::vector<uint32_t> blob_off;
        std::vector<PhaseEntry> ptab;
        std::vector<ConvSrc> csrc;
        ok = build_plan(layers, n_layers, in_c, in_h, in_w, n_classes, &plan, &blob, &blob_off, &ptab, &csrc, &bar_counts);
        if (ok) *smem_bytes = plan.smem_bytes;
    }
    *rule = ok ? 0 : g_plan_rule;
    return ok ? 1 : 0;
}

int line_build(const LayerIn *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes, LinePlan **out)
{
    *out = nullptr;
    if (!structure_ok(layers, n_layers, n_classes)) return ISC_OK;
    const isc_layer &LP = layers[n_layers - 2].d, &LF = layers[n_layers - 1].d;

    LinePlan *plan = new LinePlan();
    std::vector<uint8_t> blob, bar_counts;
    std::vector<uint32_t> blob_off;
    std::vector<PhaseEntry> ptab;
    std::vector<ConvSrc> csrc;
    if (!build_plan(layers, n_layers, in_c, in_h, in_w, n_classes, plan, &blob, &blob_off, &ptab, &csrc, &bar_counts)) {
        delete plan;
        return ISC_OK;
    }
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
    const LayerIn &MF = layers[n_layers - 1];
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
    for (size_t c = 0; c < csrc.size(); ++c) csrc[c].gmem = (unsigned long long)(plan->d_blob + blob_off[c]);
    up((void **)&plan->d_ptab, ptab.data(), ptab.size() * sizeof(PhaseEntry));
    up((void **)&plan->d_conv_src, csrc.data(), csrc.size() * sizeof(ConvSrc));
    up((void **)&plan->d_bar_counts, bar_counts.data(), bar_counts.size());
    up((void **)&plan->d_fc_w, fcw.data(), fcw.size());
    up((void **)&plan->d_fc_c, fcc.data(), fcc.size() * sizeof(FcConst));
    int32_t zero = 0;
    up((void **)&plan->d_err, &zero, sizeof(zero));
    const unsigned long long zeros4[4] = {0, 0, 0, 0};
    up((void **)&plan->d_phase_cycles, zeros4, sizeof(zeros4));
    if (cuda_ok && cudaMalloc((void **)&plan->d_dump, kSmemLimit) != cudaSuccess) cuda_ok = false;
    if (!cuda_ok) { cudaGetLastError(); line_free(plan); return ISC_ERR_NOMEM; }

    LineParams &b = plan->base;
    memset(&b, 0, sizeof(b));
    b.ptab = plan->d_ptab;
    b.conv_src = plan->d_conv_src;
    b.bar_counts = plan->d_bar_counts;
    b.n_bars = plan->n_bars;
    b.n_phases = plan->n_phases;
    b.n_conv = plan->n_conv;
    b.in_c = in_c; b.in_H = in_h; b.in_W = in_w;
    b.input_base = plan->tensor_off[0] + plan->tensors[0].line0;
    b.input_pitch16 = (uint32_t)plan->tensors[0].pitch;
    const LGeo &last = plan->tensors[(size_t)n_layers - 2];
    b.tail_base = plan->tensor_off[(size_t)n_layers - 2] + last.line0;
    b.tail_plane = last.plane_bytes; b.tail_pitch16 = (uint32_t)last.pitch; b.tail_logI = (uint32_t)ilog2(last.I);
    b.tail_C = last.C; b.tail_H = last.H; b.tail_W = last.W; b.tail_n_lines = last.n_lines;
    b.pool_mult = layers[n_layers - 2].mult[0];
    b.pool_n = 31 + layers[n_layers - 2].shift[0];
    b.pool_zp_in = LP.zp_in; b.pool_zp_out = LP.zp_out;
    b.pool_lo = LP.relu ? std::max(-128, LP.zp_out) : -128;
    b.fc_w = plan->d_fc_w; b.fc_c = plan->d_fc_c;
    b.n_classes = n_classes;
    b.err = plan->d_err;
    b.phase_cycles = plan->d_phase_cycles;
    b.stop_phase = 1 << 30;
    *out = plan;
    return ISC_OK;
}

void line_free(LinePlan *p)
{
    if (!p) return;
    cudaFree(p->d_ptab); cudaFree(p->d_conv_src); cudaFree(p->d_bar_counts); cudaFree(p->d_blob); cudaFree(p->d_fc_w);
    cudaFree(p->d_fc_c); cudaFree(p->d_err); cudaFree(p->d_phase_cycles); cudaFree(p->d_dump);
    delete p;
}

static int line_launch(LinePlan *p, LineParams &q, cudaStream_t st)
{
    if (!p->attr_set) {
        if (cudaFuncSetAttribute(k_line, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p->smem_bytes) != cudaSuccess) {
            cudaGetLastError();
            return ISC_ERR_CUDA;
        }
        p->attr_set = true;
    }
    const int grid = std::max(1, std::min(q.n_groups, p->sm_count));
    k_line<<<grid, kThreads, p->smem_bytes, st>>>(q);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess && getenv("ISC_PLAN_DEBUG")) fprintf(stderr, "line engine: launch failed: %s\n", cudaGetErrorString(e));
    return e == cudaSuccess ? ISC_OK : ISC_ERR_CUDA;
}

int line_run(LinePlan *p, const uint8_t *d_x, const NoiseStream &ns, int64_t n, int batch_hint, int32_t *d_counts,
             int8_t *d_logits, cudaStream_t st, int64_t *launches)
{
    const int64_t per_launch = batch_hint > 0 ? batch_hint : (1ll << 30);
    for (int64_t done = 0; done < n; done += per_launch) {
        const int64_t m = std::min(per_launch, n - done);
        LineParams q = p->base;
        q.x = d_x;
        q.ns = ns;
        q.ns.first_sample = ns.first_sample + done;
        q.n_samples = (int32_t)m;
        q.n_groups = (int32_t)((m + kG - 1) / kG);
        q.counts = d_counts;
        q.logits = d_logits ? d_logits + (size_t)done * p->n_classes : nullptr;
        int rc = line_launch(p, q, st);
        *launches += 1;
        if (rc) return rc;
    }
    return ISC_OK;
}

int line_check(LinePlan *p)
{
    int32_t e = 0;
    if (cudaMemcpy(&e, p->d_err, sizeof(e), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return ISC_ERR_CUDA; }
    if (e != 0) {
        if (getenv("ISC_PLAN_DEBUG")) fprintf(stderr, "line engine: wait %d on barrier %d parity %d expired in CTA %d\n", e & 0xFF, (e >> 8) & 0xFFF, (e >> 20) & 1, (int)((unsigned)e >> 21));
        cudaMemset(p->d_err, 0, sizeof(e));
        return ISC_ERR_TIMEOUT;
    }
    return ISC_OK;
}

int line_wait_probe(LinePlan *p, long long limit_ns, int32_t out[4], cudaStream_t st)
{
    if (limit_ns < 1000 || limit_ns > 100000000ll) return ISC_ERR_ARG;          // 1 us .. 100 ms
    int32_t *d_out = reinterpret_cast<int32_t *>(p->d_dump);                   // the debug read-back buffer
    k_wait_probe<<<1, 32, kCtrlBytes, st>>>(p->d_err, (unsigned long long)limit_ns, d_out);
    if (cudaGetLastError() != cudaSuccess) return ISC_ERR_CUDA;
    if (cudaMemcpyAsync(out, d_out, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ISC_ERR_CUDA; }
    return line_check(p);
}

int line_phase_cycles(LinePlan *p, unsigned long long out[4])
{
    if (cudaMemcpy(out, p->d_phase_cycles, 4 * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return ISC_ERR_CUDA;
    }
    return ISC_OK;
}

// Runs one group (samples ns.first_sample ..) up to the phase that produces `tensor` and returns that
// tensor of the first sample as [C][H][W] int32.
int line_debug_tensor(LinePlan *p, const uint8_t *d_x, const NoiseStream &ns, int tensor, int32_t *out_chw,
                      int32_t *d_counts_scratch, cudaStream_t st, int64_t *launches)
{
    if (tensor < 0 || tensor >= (int)p->tensors.size() || p->tensors[(size_t)tensor].buffer < 0) return ISC_ERR_UNSUPPORTED;
    const LGeo &t = p->tensors[(size_t)tensor];
    LineParams q = p->base;
    q.x = d_x; q.ns = ns; q.n_samples = 1; q.n_groups = 1; q.counts = d_counts_scratch; q.logits = nullptr;
    q.stop_phase = t.producer_phase;
    q.dump_off = p->tensor_off[(size_t)tensor]; q.dump_bytes = t.bytes; q.dump = p->d_dump;
    int rc = line_launch(p, q, st);
    *launches += 1;
    if (rc) return rc;
    std::vector<uint8_t> h(t.bytes);
    if (cudaMemcpyAsync(h.data(), p->d_dump, t.bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ISC_ERR_CUDA; }
    if ((rc = line_check(p))) return rc;
    for (int c = 0; c < t.C; ++c)
        for (int y = 0; y < t.H; ++y)
            for (int x = 0; x < t.W; ++x) {
                const int line = y % t.n_lines, band = y / t.n_lines;
                const size_t at = (size_t)(c / 16) * t.plane_bytes + t.line0 +
                                  ((size_t)line * t.pitch + (size_t)x * t.I + (size_t)band * 4) * 16 + (size_t)(c % 16);
                const uint8_t b = h[at];
                out_chw[((size_t)c * t.H + y) * t.W + x] = tensor == 0 ? (int32_t)b : (int32_t)(int8_t)b;
            }
    return ISC_OK;
}


}  // namespace isc
