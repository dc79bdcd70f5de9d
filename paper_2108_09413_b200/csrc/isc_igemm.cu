// Layer-by-layer implicit-GEMM convolution on the tensor cores (sm_100a): one launch per convolution over a batch of
// noisy samples, for the networks whose activations do not fit in shared memory (the 224 x 224 bottleneck network of
// the paper's second workload, Sec. 4.1).  Activations are the layer-by-layer engine's: int8, global memory,
// [sample][y][x][channel padded to 16].
//
//   D[pixel, cout] = sum over (tap, cin) of A[pixel, (tap, cin)] * W[cout, (tap, cin)]
//
// A tile is 128 output pixels x N output channels (N = 64, 128 or 256) whose int32 accumulators live in tensor
// memory.  The kernel is persistent (one CTA per SM, tiles dealt round-robin) and its warps have fixed roles that
// meet only at mbarriers:
//   * four warps gather operand rows: per reduction block (64 input channels of one filter tap) a lane issues four
//     asynchronous 16-byte copies (through L1) into the K-major core-matrix layout (four lanes read one pixel's 64 bytes) whose
//     completion arrives on the stage's barrier; a pixel outside the image is copied from a run of the input
//     zero-point kept behind the repacked weights;
//   * one thread streams the matching slices of the repacked weights with bulk copies into the same stages; for a
//     1 x 1 stride-1 layer it also brings the operand rows, one tensor copy (cp.async.bulk.tensor) per block, and
//     the gather warps idle;
//   * one thread issues two tcgen05.mma (kind::i8, K = 32) per stage and commits the stage back to the loaders;
//     accumulators alternate between two column ranges, so a tile's reduction runs under the previous one's
//     epilogue;
//   * two teams of four warps requantise (fixed-point multiplier, shift, zero-points, residual add, clamp), one
//     accumulator each: a thread owns one tile row, 32 columns per step with the next step's accumulators already
//     requested; the rows pass through a per-warp scratch area so that, every 64 columns, the results leave and the
//     next tile's residual rows arrive as contiguous runs, under the arithmetic of the following columns.
// Every wait is bounded; on expiry a role raises the CTA's abort flag and the error word, the others leave their
// loops, and the CTA frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "isc_epilogue.cuh"
#include "isc_internal.h"
#include "isc_tc.cuh"

namespace isc {

using namespace tc;

namespace {

constexpr int kTileM = 128;
constexpr int kBlockK = 64;                  // bytes of K per stage: two MMA K-steps
constexpr unsigned kHintLoad = 20000, kHintEpi = 20000, kHintMma = 20000;      // suspend-time hint of a barrier wait (ns), by role
constexpr int kMaxStages = 16;
constexpr int kStemThreads = 256;           // k_stem: two threads per tile row; two CTAs per SM (registers allow no third, nor two of 512 threads)
constexpr size_t kStemSmemLimit = 108 * 1024;          // dynamic shared memory of k_stem: two CTAs per SM
constexpr int kEpiWarps = 4, kEpiTeams = 2, kGatherWarps = 4;          // a team of epilogue warps takes every other tile
constexpr int kAllEpiWarps = kEpiWarps * kEpiTeams;
static_assert(kEpiWarps == 4, "an epilogue warp owns all N columns of its 32 rows");
constexpr int kGemmThreads = 32 * (kAllEpiWarps + kGatherWarps + 2);      // k_igemm: + the MMA warp + the weights warp
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct IgemmParams {
    alignas(64) CUtensorMap tmap_a;          // the input as (16 bytes, pixel, 16-byte column of the channels): see tma_a
    GLayer L;
    int tma_a;                               // 1 x 1 stride 1: the operand rows arrive by one tensor copy per block, the gather warps idle
    int batch, n_tile, tmem_cols, stages;
    uint32_t scratch_off;                    // the epilogue warps' row scratch within the dynamic shared memory
    uint32_t m_total, tiles_m;               // batch * hout * wout (< 2^31); tiles of 128 of them
    const int8_t *in, *res;
    int8_t *out;
    const int8_t *wpack;                     // [cout tile][tap][cin block][4 K columns][n_tile rows][16 bytes]
    const int4 *cst;                         // per output channel: folded bias, multiplier, rounding addend, shift - 1
    int fast_requant, fast_residual, lo;     // every shift >= 2; residual rescale by 2^-31 or 2^-32; lower clamp
    uint32_t res_m2, res_k8;                 // residual multiplier and addend in the 2^-32 form; offset of the two-instruction form
    int res_short;                           // the two-instruction form reproduces the residual term (see requant16_fast)
    int debug_stall;                         // test hook: the weights are never sent, so every wait of the kernel runs out
    long long res_r2;
    int32_t *err;
};

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

__device__ __forceinline__ long long mul_wide(int a, int b)
{
    long long d;
    asm("mul.wide.s32 %0, %1, %2;" : "=l"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ long long mad_wide_u(uint32_t a, uint32_t b, long long c)
{
    long long d;
    asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(d) : "r"(a), "r"(b), "l"(c));
    return d;
}

// 16 accumulators -> 16 int8 outputs with 32-bit arithmetic.  With s = shift - 1 >= 1,
//   rs((acc + bias) * mult, 31 + shift) + zp_out = (hi32((acc + bias) * mult) + c) >> s,  c = 2^(s-1) + zp_out * 2^s,
// exactly (the rounding half 2^(31+s) is a multiple of 2^32, so the product's low word cannot change the floor), and
//   rs((r - zp_res) * res_mult, n) = hi32(u * m2 + R2),  u = r + 128, m2 = res_mult * 2^(32-n), n = 31 or 32,
// with R2 = (2^(n-1) - (128 + zp_res) * res_mult) * 2^(32-n) (kRes = 1).  kRes = 2 is the same term without the
// 64-bit addend: hi32((256 k + u) * m2) - c_r for an offset k that the host has checked on all 256 values of u
// (residual_short_form); 256 k is merged into u by the byte permute that extracts u, and c_r is folded into c.
// `cst` points at this block's constants in shared memory.
template <int kRes>
__device__ __forceinline__ uint4 requant16_fast(const int *acc, uint32_t cst, uint4 rv, uint32_t m2, long long r2, uint32_t k8, int lo)
{
    const uint32_t rw[4] = {rv.x ^ 0x80808080u, rv.y ^ 0x80808080u, rv.z ^ 0x80808080u, rv.w ^ 0x80808080u};
    uint32_t packed[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        int y[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            int4 c;
            asm("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(c.x), "=r"(c.y), "=r"(c.z), "=r"(c.w) : "r"(cst + (4 * g + k) * 16));
            int v = (hi32(mul_wide(acc[4 * g + k] + c.x, c.y)) + c.z) >> c.w;
            if (kRes == 1) v += hi32(mad_wide_u(__byte_perm(rw[g], 0u, 0x4440u | (uint32_t)k), m2, r2));
            if (kRes == 2) v += hi32(mad_wide_u(__byte_perm(rw[g], k8, 0x7650u | (uint32_t)k), m2, 0ll));
            y[k] = max(v, lo);
        }
        packed[g] = pack4_sat(y[0], y[1], y[2], y[3]);
    }
    return make_uint4(packed[0], packed[1], packed[2], packed[3]);
}

// 32 accumulator columns of this thread's lane, asynchronously; the registers are valid after tmem_ld32_wait(),
// which names them so that no use can move above it
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, int (&v)[2][16])
{
    tmem_ld16_issue(taddr, v[0]);
    tmem_ld16_issue(taddr + 16u, v[1]);
}
__device__ __forceinline__ void tmem_ld32_wait(int (&v)[2][16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0][0]), "+r"(v[0][1]), "+r"(v[0][2]), "+r"(v[0][3]), "+r"(v[0][4]), "+r"(v[0][5]), "+r"(v[0][6]), "+r"(v[0][7]),
                   "+r"(v[0][8]), "+r"(v[0][9]), "+r"(v[0][10]), "+r"(v[0][11]), "+r"(v[0][12]), "+r"(v[0][13]), "+r"(v[0][14]), "+r"(v[0][15]),
                   "+r"(v[1][0]), "+r"(v[1][1]), "+r"(v[1][2]), "+r"(v[1][3]), "+r"(v[1][4]), "+r"(v[1][5]), "+r"(v[1][6]), "+r"(v[1][7]),
                   "+r"(v[1][8]), "+r"(v[1][9]), "+r"(v[1][10]), "+r"(v[1][11]), "+r"(v[1][12]), "+r"(v[1][13]), "+r"(v[1][14]), "+r"(v[1][15])
                 :: "memory");
}

// Bounded wait for a phase of an mbarrier; false after the limit (the caller raises the error word).
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity)
{
    if (mbar_test(bar, parity)) return true;
    const unsigned long long t0 = globaltimer();
    for (int spin = 0;; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 7) == 7 && globaltimer() - t0 > kWaitLimitNs) return false;
    }
}
// The same for the roles of k_igemm, which also give up when another role has raised the CTA's abort flag.  With
// `kHintNs` the wait is parked in hardware for up to that long per attempt instead of polling (the abort flag and
// the time limit are looked at every eighth attempt).
template <unsigned kHintNs>
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const volatile int *abort_flag)
{
    if (mbar_test(bar, parity)) return true;
    const unsigned long long t0 = globaltimer();
    for (int spin = 0;; ++spin) {
        if (kHintNs) {
            // parked in hardware until the phase completes or the hint runs out
            uint32_t done;
            asm volatile("{\n\t.reg .pred p;\n\t"
                         "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
                         "selp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(done) : "r"(bar), "r"(parity), "r"(kHintNs) : "memory");
            if (done) return true;
        } else if (mbar_try(bar, parity)) {
            return true;
        }
        if ((spin & 7) == 7 && (*abort_flag || globaltimer() - t0 > kWaitLimitNs)) return false;
    }
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// the same through L1: the taps of a 3 x 3 filter read a pixel's row nine times, and every CTA reads the zero-point run
__device__ __forceinline__ void cp_async16_cached(uint32_t dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// one arrival on `bar` (counted in its initial count) once every cp.async this thread has issued so far is complete
__device__ __forceinline__ void cp_async_arrive(uint32_t bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// all of this thread's copy groups but the newest are complete
__device__ __forceinline__ void cp_async_wait_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// A stage ring position: index and how many times the ring has wrapped.
struct Ring {
    int s = 0, use = 0;
    __device__ __forceinline__ void advance(int stages) { if (++s == stages) { s = 0; ++use; } }
};

// What an epilogue warp needs from the kernel's prologue.
struct EpiCtx {
    uint32_t sbase, tmem, n_tiles, grid_n;
    int tiles_n, warp, lane;
    uint32_t cst_s, acc_full, acc_free;       // shared-memory addresses: constants, the two accumulators' barriers
    const volatile int *abort_flag;
};

// The epilogue of k_igemm.  Warp w owns lanes 32 (w mod 4) .. +31 of an accumulator (= 32 tile rows) and all N
// columns; team w / 4 takes every other tile of the CTA (accumulator `team`).  A thread requantises its own row in
// place in a per-warp scratch area in shared memory (row stride N + 16 bytes: conflict-free for the row-wise and
// for the coalesced access).  After every 64 columns the warp writes those columns of its 32 rows out as runs of
// 64 contiguous bytes per row and requests the same columns of the residual rows of its next tile into the
// space that has just been read, so memory traffic runs under the arithmetic of the following columns.
// kMode 0: 64-bit requantisation (any shift), 1: 32-bit form, 2 / 3: 32-bit form with the residual add (3: its
// two-instruction form).
template <int kMode>
__device__ __forceinline__ bool epilogue_role(const IgemmParams &p, const EpiCtx &c)
{
    const GLayer &L = p.L;
    const int warp = c.warp, lane = c.lane, n_tile = p.n_tile, tiles_n = c.tiles_n;
    const int q = warp & 3, team = warp / kEpiWarps;
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const uint32_t row_stride = (uint32_t)n_tile + 16u;
    const uint32_t scr0 = c.sbase + p.scratch_off + (uint32_t)warp * 32u * row_stride;
    const uint32_t scr_row = scr0 + (uint32_t)lane * row_stride;
    // coalesced access to 64 columns of the 32 rows: four lanes per row, eight rows per instruction
    const int crow = lane >> 2, cchunk = lane & 3;
    const uint32_t scr_co = scr0 + (uint32_t)crow * row_stride + (uint32_t)cchunk * 16u;
    const size_t co_step = (size_t)8 * L.coutp;
    // where tile t's rows start in the output / residual tensors, for this lane's coalesced position; null when the
    // row is beyond the last pixel (the rows of a warp that are valid are its first ones)
    auto tile_ptr = [&](const int8_t *base, uint32_t t, uint32_t &rows) {
        const uint32_t m_idx = t / (uint32_t)tiles_n;
        const uint32_t m0 = m_idx * kTileM + (uint32_t)q * 32u;
        rows = m0 < p.m_total ? min(32u, p.m_total - m0) : 0u;
        return base + (size_t)(m0 + (uint32_t)crow) * L.coutp + (int)(t - m_idx * tiles_n) * n_tile + cchunk * 16;
    };
    auto residual_fetch = [&](const int8_t *src, uint32_t rows, int c0) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if ((uint32_t)(8 * k + crow) < rows) cp_async16(scr_co + (uint32_t)(8 * k) * row_stride + (uint32_t)c0, src + (size_t)k * co_step + c0);
    };
    // the team's tiles: every kEpiTeams-th of the CTA's
    const uint32_t t_step = (uint32_t)kEpiTeams * c.grid_n;
    uint32_t t = blockIdx.x + (uint32_t)team * c.grid_n;
    if (kMode >= 2 && t < c.n_tiles) {
        uint32_t rows;
        const int8_t *src = tile_ptr(p.res, t, rows);
        for (int c0 = 0; c0 < n_tile; c0 += 64) residual_fetch(src, rows, c0);
    }
    for (int au = 0; t < c.n_tiles; t += t_step, ++au) {
        const uint32_t m_idx = t / (uint32_t)tiles_n;
        const int n0 = (int)(t - m_idx * tiles_n) * n_tile;
        const uint32_t m = m_idx * kTileM + (uint32_t)q * 32u + (uint32_t)lane;
        const int8_t *res_px = (kMode == 0 && p.res && m < p.m_total) ? p.res + (size_t)m * L.coutp : nullptr;
        uint32_t rows, rows_next = 0;
        int8_t *dst = const_cast<int8_t *>(tile_ptr(p.out, t, rows));
        const int8_t *res_next = (kMode >= 2 && t + t_step < c.n_tiles) ? tile_ptr(p.res, t + t_step, rows_next) : nullptr;
        cp_async_wait_all();                                        // the tile's residual rows, requested during the previous tile
        __syncwarp();
        if (!wait_bar<kHintEpi>(c.acc_full + 8u * (uint32_t)team, (uint32_t)au & 1u, c.abort_flag)) {
            cp_async_wait_all();                                    // the next tile's residual rows may still be landing
            return false;
        }
        tc_fence_after();
        const uint32_t acc_base = c.tmem + lane_base + (uint32_t)(team * n_tile);
        const uint32_t cst0 = c.cst_s + (uint32_t)n0 * 16u;
        // 32 columns per step, the accumulators of the next step requested before this step's arithmetic
        auto step = [&](int (&acc)[2][16], int c0) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int cc = c0 + 16 * h;
                uint4 v;
                if (kMode == 3) {
                    v = requant16_fast<2>(acc[h], cst0 + (uint32_t)cc * 16u, ld_shared_v4(scr_row + (uint32_t)cc), p.res_m2, 0ll, p.res_k8, p.lo);
                } else if (kMode == 2) {
                    v = requant16_fast<1>(acc[h], cst0 + (uint32_t)cc * 16u, ld_shared_v4(scr_row + (uint32_t)cc), p.res_m2, p.res_r2, 0u, p.lo);
                } else if (kMode == 1) {
                    v = requant16_fast<0>(acc[h], cst0 + (uint32_t)cc * 16u, make_uint4(0, 0, 0, 0), 0u, 0ll, 0u, p.lo);
                } else {
#pragma unroll
                    for (int o = 0; o < 16; ++o) acc[h][o] += __ldg(L.bias + n0 + cc + o);
                    v = epilogue16(acc[h], L, n0 + cc, res_px);
                }
                st_shared_v4(scr_row + (uint32_t)cc, v);
            }
        };
        int acc_a[2][16], acc_b[2][16];
        tmem_ld32_issue(acc_base, acc_a);
#pragma unroll 1
        for (int c0 = 0; c0 < n_tile; c0 += 64) {                   // N is a multiple of 64
            tmem_ld32_wait(acc_a);
            tmem_ld32_issue(acc_base + (uint32_t)c0 + 32u, acc_b);
            step(acc_a, c0);
            tmem_ld32_wait(acc_b);
            if (c0 + 64 < n_tile) {
                tmem_ld32_issue(acc_base + (uint32_t)c0 + 64u, acc_a);
            } else {
                tc_fence_before();
                mbar_arrive(c.acc_free + 8u * (uint32_t)team);      // the accumulator is in registers: the next tile may overwrite it
            }
            step(acc_b, c0 + 32);
            __syncwarp();
            uint4 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) v[k] = ld_shared_v4(scr_co + (uint32_t)(8 * k) * row_stride + (uint32_t)c0);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if ((uint32_t)(8 * k + crow) < rows) *reinterpret_cast<uint4 *>(dst + (size_t)k * co_step + c0) = v[k];
            __syncwarp();
            if (res_next) residual_fetch(res_next, rows_next, c0);
        }
    }
    cp_async_wait_all();
    return true;
}

__global__ void __launch_bounds__(kGemmThreads, 1) k_igemm(const __grid_constant__ IgemmParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];            // operand stages | requantisation constants | epilogue scratch
    __shared__ unsigned long long bar_full[kMaxStages], bar_free[kMaxStages], bar_acc_full[2], bar_acc_free[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int abort_s;
    const GLayer &L = p.L;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    const int n_tile = p.n_tile, stages = p.stages;
    const uint32_t a_bytes = kTileM * kBlockK, b_bytes = (uint32_t)n_tile * kBlockK, stage_bytes = a_bytes + b_bytes;
    int4 *cst_s = reinterpret_cast<int4 *>(smem + (size_t)stages * stage_bytes);
    if (tid == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(smem_u32(&bar_full[s]), p.tma_a ? 1 : kGatherWarps * 32 + 1); mbar_init(smem_u32(&bar_free[s]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bar_acc_full[i]), 1); mbar_init(smem_u32(&bar_acc_free[i]), kEpiWarps * 32); }
        abort_s = 0;
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_base_s), (uint32_t)p.tmem_cols);
    for (int i = tid; i < L.coutp; i += kGemmThreads) cst_s[i] = __ldg(p.cst + i);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;

    // tiles in m-major order (the CTAs of one wave share operand rows in L2), dealt round-robin to the CTAs
    const int tiles_n = L.coutp / n_tile;
    const uint32_t n_tiles = p.tiles_m * (uint32_t)tiles_n, grid_n = gridDim.x;
    const int cblocks = L.cinp / kBlockK, nkb = L.kh * L.kw * cblocks;
    bool ok = true;

    if (warp < kAllEpiWarps) {
        EpiCtx c;
        c.sbase = sbase; c.tmem = tmem; c.n_tiles = n_tiles; c.grid_n = grid_n; c.tiles_n = tiles_n; c.warp = warp; c.lane = lane;
        c.cst_s = smem_u32(cst_s);
        c.acc_full = smem_u32(&bar_acc_full[0]); c.acc_free = smem_u32(&bar_acc_free[0]);
        c.abort_flag = &abort_s;
        const bool fast = p.fast_requant && (!p.res || p.fast_residual);
        if (fast && p.res && p.res_short) ok = epilogue_role<3>(p, c);
        else if (fast && p.res) ok = epilogue_role<2>(p, c);
        else if (fast) ok = epilogue_role<1>(p, c);
        else ok = epilogue_role<0>(p, c);
    } else if (warp < kAllEpiWarps + kGatherWarps) {
        // ---- operand rows: per reduction block a warp copies 32 tile rows x 64 bytes with four asynchronous 16-byte
        // copies per lane (lane = 16-byte column x row within a group of eight, so that an instruction reads whole
        // 64-byte rows) whose completion arrives on the stage's barrier.  A row outside the image is copied from a
        // 64-byte run of the input zero-point that follows the repacked weights, so every row takes the same path.
        const int gw = warp - kAllEpiWarps, chunk = lane & 3, rsub = lane >> 2;
        const int8_t *zp_src = p.wpack + (size_t)L.coutp * (size_t)(L.kh * L.kw) * (size_t)L.cinp + chunk * 16;
        const int8_t *in_c = p.in + chunk * 16;
        // K-major core matrices: 16-byte column j of row r at j * (128 rows * 16) + r * 16
        const uint32_t dst0 = sbase + (uint32_t)chunk * 2048u + (uint32_t)(32 * gw + rsub) * 16u;
        Ring ring;
        const uint32_t px_per_sample = (uint32_t)(L.hout * L.wout);
        for (uint32_t t = blockIdx.x; t < n_tiles && ok && !p.tma_a; t += grid_n) {
            const uint32_t m0 = (t / (uint32_t)tiles_n) * kTileM + (uint32_t)(32 * gw + rsub);
            int iy0[4], ix0[4], off[4];                         // this lane's four rows: 8 apart
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t m = m0 + 8u * (uint32_t)i;
                const bool valid = m < p.m_total;
                const uint32_t mm = valid ? m : 0u;
                const uint32_t b = mm / px_per_sample, pp = mm - b * px_per_sample;
                const int oy = (int)(pp / (uint32_t)L.wout), ox = (int)pp - oy * L.wout;
                iy0[i] = valid ? oy * L.stride - L.pad : -0x100000;             // an invalid row is outside for every tap
                ix0[i] = ox * L.stride - L.pad;
                off[i] = (((int)b * L.hin + oy * L.stride - L.pad) * L.win + ix0[i]) * L.cinp;    // the tensor is < 2^31 bytes
            }
            for (int tap = 0, r = 0, sx = 0; tap < L.kh * L.kw && ok; ++tap, sx = (sx + 1 == L.kw) ? 0 : sx + 1, r += (sx == 0)) {
                const int tap_off = (r * L.win + sx) * L.cinp;
                bool inside[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) inside[i] = (unsigned)(iy0[i] + r) < (unsigned)L.hin && (unsigned)(ix0[i] + sx) < (unsigned)L.win;
                for (int cb = 0; cb < cblocks; ++cb, ring.advance(stages)) {
                    if (ring.use >= 1) {
                        ok = wait_bar<kHintLoad>(smem_u32(&bar_free[ring.s]), (uint32_t)(ring.use - 1) & 1u, &abort_s);
                        if (!ok) break;
                    }
                    const uint32_t dst = dst0 + (uint32_t)ring.s * stage_bytes;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        cp_async16_cached(dst + (uint32_t)i * 128u, inside[i] ? in_c + (off[i] + tap_off + cb * kBlockK) : zp_src);
                    }
                    cp_async_arrive(smem_u32(&bar_full[ring.s]));
                }
            }
        }
        cp_async_wait_all();
    } else if (warp == kAllEpiWarps + kGatherWarps) {
        // ---- one thread issues the MMAs: two K-steps per stage, accumulators alternate between two column ranges
        if (lane == 0) {
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_tile >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
            Ring ring;
            int j = 0;
            for (uint32_t t = blockIdx.x; t < n_tiles && ok; t += grid_n, ++j) {
                const int buf = j & 1, au = j >> 1;
                if (au >= 1) {
                    ok = wait_bar<kHintMma>(smem_u32(&bar_acc_free[buf]), (uint32_t)(au - 1) & 1u, &abort_s);
                    if (!ok) break;
                }
                for (int kb = 0; kb < nkb; ++kb, ring.advance(stages)) {
                    ok = wait_bar<kHintMma>(smem_u32(&bar_full[ring.s]), (uint32_t)ring.use & 1u, &abort_s);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t stage = sbase + (uint32_t)ring.s * stage_bytes;
#pragma unroll
                    for (int k2 = 0; k2 < 2; ++k2) {
                        const uint64_t ad = make_desc(stage + (uint32_t)k2 * 4096u, 2048u, 128u);
                        const uint64_t bd = make_desc(stage + a_bytes + (uint32_t)k2 * 2u * (uint32_t)n_tile * 16u, (uint32_t)n_tile * 16u, 128u);
                        mma_i8(tmem + (uint32_t)(buf * n_tile), ad, bd, idesc, (kb > 0 || k2 > 0) ? 1u : 0u);
                    }
                    commit_to(smem_u32(&bar_free[ring.s]));
                }
                if (ok) commit_to(smem_u32(&bar_acc_full[buf]));
            }
        }
        __syncwarp();
    } else {
        // ---- one thread streams the repacked weights: one bulk copy per block into the stage's second part
        if (lane == 0 && !p.debug_stall) {
            Ring ring;
            for (uint32_t t = blockIdx.x; t < n_tiles && ok; t += grid_n) {
                const int8_t *wtile = p.wpack + (size_t)(t % tiles_n) * (size_t)nkb * b_bytes;
                for (int kb = 0; kb < nkb; ++kb, ring.advance(stages)) {
                    if (ring.use >= 1) {
                        ok = wait_bar<kHintLoad>(smem_u32(&bar_free[ring.s]), (uint32_t)(ring.use - 1) & 1u, &abort_s);
                        if (!ok) break;
                    }
                    mbar_expect_tx(smem_u32(&bar_full[ring.s]), p.tma_a ? a_bytes + b_bytes : b_bytes);
                    if (p.tma_a) {
                        // box {16 bytes, 128 pixels, 4 columns} of the 3-D view lands as [column][pixel][16 bytes], which is
                        // the K-major core-matrix layout; pixels beyond the last one are filled with zeros and never stored
                        asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                                     ::"r"(sbase + (uint32_t)ring.s * stage_bytes), "l"(reinterpret_cast<uint64_t>(&p.tmap_a)), "r"(0),
                                       "r"((int)((t / (uint32_t)tiles_n) * kTileM)), "r"(kb * 4), "r"(smem_u32(&bar_full[ring.s])) : "memory");
                    }
                    bulk_g2s(sbase + (uint32_t)ring.s * stage_bytes + a_bytes, wtile + (size_t)kb * b_bytes, b_bytes, smem_u32(&bar_full[ring.s]));
                }
            }
            if (!ok) {
                // copies already issued may still be landing in this CTA's shared memory: give them time before the exit
                const unsigned long long t0 = globaltimer();
                while (globaltimer() - t0 < 50000ull) __nanosleep(1000);
            }
        }
        __syncwarp();
    }
    if (!ok) {
        if (!abort_s) atomicCAS(p.err, 0, 1 + (int)blockIdx.x);
        abort_s = 1;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) tmem_dealloc(tmem, (uint32_t)p.tmem_cols);
}


// ------------------------------------------------------------------ first convolution on the tensor cores
//
// The stem of a network whose input is the noisy image (Def. 3.4): a k x k convolution over <= 4 input channels.
// One CTA = one sample x one band of output rows.  The band's input rows are drawn (Philox -> inverse-CDF table ->
// add -> saturate to 0..255, Def. 3.3 / Eq. 2) into a shared-memory patch as 4 bytes per pixel, padded with the input
// zero-point, and never written to memory.  The GEMM takes one filter row per K-step: eight horizontally adjacent
// pixels x 4 bytes = 32 bytes of K (pixels beyond the filter width meet zero weights), so a tile of 128 output pixels
// is `kh` MMAs.  Each thread copies its pixel's `kh` windows from the patch into the K-major operand stage; tiles
// alternate between two stages and two halves of the accumulator columns, so the requantisation of one tile runs
// while the MMAs of the next are in flight.
struct StemParams {
    GLayer L;
    int in_c, band_rows, n_bands, tiles_per_band, tmem_cols;
    uint32_t patch_bytes, w_bytes;
    uint32_t tab_off;                        // the noise tables' copy in shared memory (after the patch), 0: searched in global memory
    const uint8_t *x;                        // clean image, CHW
    NoiseStream ns;
    const int8_t *wpack;                     // [filter row][2 K columns][coutp rows][16 bytes]
    const int4 *cst;
    int fast_requant, lo;
    int8_t *out;
    int32_t *err;
};

__global__ void __launch_bounds__(kStemThreads, 2) k_stem(const __grid_constant__ StemParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ unsigned long long bar_w, bar_full[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int abort_s;
    __shared__ __align__(16) int4 cst_s[256];
    const GLayer &L = p.L;
    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t sbase = smem_u32(smem);
    const int N = L.coutp, kh = L.kh;
    const uint32_t a_bytes = (uint32_t)kh * kTileM * 32u;
    const uint32_t w_off = 0, a_off = p.w_bytes, patch_off = a_off + 2u * a_bytes;        // weights | two operand stages | patch
    if (tid == 0) {
        mbar_init(smem_u32(&bar_w), 1);
        mbar_init(smem_u32(&bar_full[0]), 1);
        mbar_init(smem_u32(&bar_full[1]), 1);
        abort_s = 0;
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_base_s), (uint32_t)p.tmem_cols);
    for (int i = tid; i < N; i += kStemThreads) cst_s[i] = __ldg(p.cst + i);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    if (tid == 0) {
        mbar_expect_tx(smem_u32(&bar_w), p.w_bytes);
        bulk_g2s(sbase + w_off, p.wpack, p.w_bytes, smem_u32(&bar_w));
    }

    // ---- the band's noisy input rows
    const int b = blockIdx.y;
    const int64_t j = p.ns.first_sample + b;
    const int oy0 = blockIdx.x * p.band_rows, oy1 = min(L.hout, oy0 + p.band_rows);
    const int wpad = L.win + 2 * L.pad + 8;                     // 8 more pixels: the windows of the last columns stay inside
    const int iy0 = oy0 * L.stride - L.pad;
    const int rows_in = (oy1 - oy0 - 1) * L.stride + kh;
    uint32_t *patch = reinterpret_cast<uint32_t *>(smem + patch_off);
    const uint32_t zp_fill = (uint32_t)(L.zp_in & 0xFF) * (0x01010101u >> (8 * (4 - p.in_c)));
    for (int i = tid; i < rows_in * wpad; i += kStemThreads) patch[i] = zp_fill;
    if (p.tab_off && p.ns.guide) {
        // cumulative table, then the guide table that follows it in memory
        uint32_t *tab = reinterpret_cast<uint32_t *>(smem + p.tab_off);
        for (int i = tid; i < 2 * p.ns.T + 1 + kNoiseGuide + 1; i += kStemThreads) tab[i] = __ldg(p.ns.cum + i);
    }
    __syncthreads();
    const int vy0 = max(0, iy0), vy1 = min(L.hin, iy0 + rows_in);
    if (vy1 > vy0) {
        uint8_t *pb = reinterpret_cast<uint8_t *>(patch);
        const uint32_t ctr3 = p.ns.ctr3_fixed | (uint32_t)(((j >> 32) & 0xFF) << 8);
        const uint32_t ctr1 = (uint32_t)(j & 0xFFFFFFFFll);
        if ((L.win & 3) == 0 && p.ns.guide) {
            // every Philox block (four consecutive elements of the CHW order) lies within one image row: a thread
            // takes whole blocks, all channels of the band's rows as one index space, the four searches interleaved
            const int qpr = L.win >> 2, qpc = (vy1 - vy0) * qpr;
            for (int i = tid; i < p.in_c * qpc; i += kStemThreads) {
                const int c = i / qpc, ic = i - c * qpc;
                const int hr = ic / qpr, wq = ic - hr * qpr;
                const int h = vy0 + hr;
                const uint32_t e = (uint32_t)((c * L.hin + h) * L.win) + 4u * (uint32_t)wq;
                const uint4 r = philox4x32_10(make_uint4(e >> 2, ctr1, p.ns.ctr2, ctr3), p.ns.key0, p.ns.key1);
                const uint32_t clean = __ldg(reinterpret_cast<const uint32_t *>(p.x + e));
                int z[4];
                if (p.tab_off) noise_levels4_shared(r, sbase + p.tab_off, sbase + p.tab_off + 4u * (uint32_t)(2 * p.ns.T + 1), p.ns.T, p.ns.guide_steps, z);
                else noise_levels4(r, p.ns.cum, p.ns.guide, p.ns.T, p.ns.guide_steps, z);
                uint8_t *dst = pb + ((h - iy0) * wpad + (4 * wq + L.pad)) * 4 + c;
#pragma unroll
                for (int k = 0; k < 4; ++k) dst[4 * k] = (uint8_t)min(255, max(0, (int)((clean >> (8 * k)) & 0xFFu) + z[k]));
            }
        } else {
            for (int c = 0; c < p.in_c; ++c) {
                const int64_t e_begin = ((int64_t)c * L.hin + vy0) * L.win, e_end = ((int64_t)c * L.hin + vy1) * L.win;
                for (int64_t q = (e_begin >> 2) + tid; q < ((e_end + 3) >> 2); q += kStemThreads) {
                    const uint4 r = philox4x32_10(make_uint4((uint32_t)q, ctr1, p.ns.ctr2, ctr3), p.ns.key0, p.ns.key1);
                    const uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int64_t e = q * 4 + k;
                        if (e < e_begin || e >= e_end) continue;
                        const int rem = (int)(e - (int64_t)c * L.hin * L.win);
                        const int h = rem / L.win, w = rem - h * L.win;
                        int v = (int)__ldg(p.x + e) + (p.ns.guide ? noise_level_guided(u[k], p.ns.cum, p.ns.guide, p.ns.T) : noise_level(u[k], p.ns.cum, p.ns.T));
                        v = min(255, max(0, v));
                        pb[((h - iy0) * wpad + (w + L.pad)) * 4 + c] = (uint8_t)v;
                    }
                }
            }
        }
    }
    __syncthreads();

    // ---- tiles of 128 output pixels of the band.  Thread = tile row `px` x one of kStemThreads / 128 groups: the
    // groups share the filter rows' windows and the 16-channel chunks round-robin.
    const int band_px = (oy1 - oy0) * L.wout;
    const int n_tiles = (band_px + kTileM - 1) / kTileM;
    const uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
    const int px_row = tid & (kTileM - 1), grp = tid >> 7;
    bool ok = true;
    if (tid == 0) ok = wait_bar(smem_u32(&bar_w), 0);
    for (int t = 0; t <= n_tiles; ++t) {
        if (t < n_tiles) {
            // operand stage of tile t: free once the MMAs of tile t - 2 are complete (waited for by its epilogue below)
            const uint32_t stage = sbase + a_off + (uint32_t)(t & 1) * a_bytes;
            const int px = t * kTileM + px_row;
            const int pp = px < band_px ? px : 0;
            const int oyl = pp / L.wout, ox = pp - oyl * L.wout;
            for (int r = grp; r < kh; r += kStemThreads / kTileM) {
                const uint32_t *src = patch + (oyl * L.stride + r) * wpad + ox * L.stride;
                st_shared_v4(stage + (uint32_t)r * 4096u + 0u * 2048u + px_row * 16, make_uint4(src[0], src[1], src[2], src[3]));
                st_shared_v4(stage + (uint32_t)r * 4096u + 1u * 2048u + px_row * 16, make_uint4(src[4], src[5], src[6], src[7]));
            }
            fence_proxy_async();
        }
        __syncthreads();
        if (t < n_tiles && tid == 0) {
            tc_fence_after();
            if (ok && !abort_s) {
                const uint32_t stage = sbase + a_off + (uint32_t)(t & 1) * a_bytes;
                for (int r = 0; r < kh; ++r) {
                    const uint64_t ad = make_desc(stage + (uint32_t)r * 4096u, 2048u, 128u);
                    const uint64_t bd = make_desc(sbase + w_off + (uint32_t)r * 2u * (uint32_t)N * 16u, (uint32_t)N * 16u, 128u);
                    mma_i8(tmem + (uint32_t)(t & 1) * (uint32_t)N, ad, bd, idesc, r > 0 ? 1u : 0u);
                }
            }
            commit_to(smem_u32(&bar_full[t & 1]));
        }
        if (t >= 1) {
            // epilogue of tile t - 1 while the MMAs of tile t run
            const int tt = t - 1;
            if (ok && !abort_s) ok = wait_bar(smem_u32(&bar_full[tt & 1]), (uint32_t)(tt >> 1) & 1u);
            if (!ok) abort_s = 1;
            tc_fence_after();
            const int px = tt * kTileM + px_row;
            const bool valid = px < band_px;
            const size_t m = ((size_t)b * L.hout + oy0) * L.wout + (size_t)(valid ? px : 0);
            for (int c0 = 16 * grp; c0 < N; c0 += 16 * (kStemThreads / kTileM)) {
                int acc[16];
                tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(tt & 1) * (uint32_t)N + (uint32_t)c0, acc);
                if (valid && !abort_s) {
                    uint4 v;
                    if (p.fast_requant) {
                        v = requant16_fast<0>(acc, smem_u32(cst_s + c0), make_uint4(0, 0, 0, 0), 0u, 0ll, 0u, p.lo);
                    } else {
#pragma unroll
                        for (int o = 0; o < 16; ++o) acc[o] += __ldg(L.bias + c0 + o);
                        v = epilogue16(acc, L, c0, nullptr);
                    }
                    *reinterpret_cast<uint4 *>(p.out + m * L.coutp + c0) = v;
                }
            }
            tc_fence_before();
        }
    }
    if (!ok) atomicCAS(p.err, 0, 1 + (int)blockIdx.x);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) tmem_dealloc(tmem, (uint32_t)p.tmem_cols);
}

}  // namespace

// ------------------------------------------------------------------ host side

int igemm_tile_n(const GLayer &G)
{
    if ((G.op != ISC_CONV2D && G.op != ISC_FC) || G.cinp % kBlockK != 0 || G.cin != G.cinp) return 0;
    if (G.coutp % 256 == 0) return 256;
    if (G.coutp % 128 == 0) return 128;
    if (G.coutp % 64 == 0) return 64;
    return 0;
}

// the repacked weights, then 64 bytes of the input zero-point (the operand row of a pixel outside the image)
size_t igemm_pack_bytes(const GLayer &G)
{
    return (size_t)G.coutp * (size_t)(G.kh * G.kw) * (size_t)G.cinp + kBlockK;
}

// w: [cout][cin][kh][kw] as the model gives it -> [cout tile][tap][cin block][4 columns of 16 channels][n_tile rows][16]
void igemm_pack_weights(const GLayer &G, const int8_t *w, int8_t *out)
{
    const int n_tile = igemm_tile_n(G), taps = G.kh * G.kw, cblocks = G.cinp / kBlockK;
    size_t at = 0;
    for (int t = 0; t < G.coutp / n_tile; ++t)
        for (int tap = 0; tap < taps; ++tap)
            for (int cb = 0; cb < cblocks; ++cb)
                for (int j = 0; j < 4; ++j)
                    for (int n = 0; n < n_tile; ++n)
                        for (int e = 0; e < 16; ++e, ++at) {
                            const int oc = t * n_tile + n, ci = cb * kBlockK + j * 16 + e;
                            out[at] = (oc < G.cout && ci < G.cin) ? w[((size_t)oc * G.cin + ci) * taps + tap] : (int8_t)0;
                        }
    for (int e = 0; e < kBlockK; ++e) out[at + e] = (int8_t)G.zp_in;
}

// The residual term F(u) = floor((u * m2 + R2) / 2^32), u = r + 128 in 0..255 (see requant16_fast), as
// hi32((256 k + u) * m2) - c: the smallest k < 4096 for which the two agree on all 256 inputs, or false.
bool residual_short_form(int res_mult, int res_shift, int zp_res, uint32_t *k8, int32_t *c_out)
{
    const int n = 31 - res_shift;
    if (n != 31 && n != 32) return false;
    if (res_mult <= 0) return false;
    const uint64_t m2 = (uint64_t)(uint32_t)res_mult << (32 - n);
    if (m2 >= (1ull << 32)) return false;
    const int64_t r2 = ((1ll << (n - 1)) - (128ll + zp_res) * (int64_t)res_mult) * (1ll << (32 - n));
    for (uint32_t k = 0; k < 4096; ++k) {
        int64_t c = 0;
        bool same = true;
        for (uint32_t u = 0; u < 256 && same; ++u) {
            const int64_t want = ((int64_t)(u * m2) + r2) >> 32;                 // arithmetic shift: floor
            const int64_t got = (int64_t)(((uint64_t)(256u * k + u) * m2) >> 32);
            if (u == 0) c = got - want;
            same = got - want == c;
        }
        if (same) { *k8 = k << 8; *c_out = (int32_t)c; return true; }
    }
    return false;
}

// Per output channel {folded bias, multiplier, rounding addend, shift - 1}; returns whether every shift is >= 2 (the
// condition of the 32-bit form).  `bias_folded`, `mult`, `shift` are the layer's host arrays padded to coutp.  For a
// layer with a residual operand whose term has the two-instruction form, that form's constant is folded into the
// rounding addends and *res_k8 is its offset; otherwise *res_k8 = 0xFFFFFFFF.
bool igemm_constants(const GLayer &G, const int32_t *bias_folded, const int32_t *mult, const int32_t *shift, int32_t *out4,
                     bool has_residual, uint32_t *res_k8)
{
    bool fast = true;
    for (int o = 0; o < G.coutp; ++o) fast = fast && shift[o] - 1 >= 1;
    uint32_t k8 = 0;
    int32_t c_res = 0;
    bool short_form = fast && has_residual && residual_short_form(G.res_mult, G.res_shift, G.zp_res, &k8, &c_res);
    for (int o = 0; o < G.coutp && short_form; ++o) {
        const int s = shift[o] - 1;
        const long long add = (1ll << (s - 1)) + ((long long)G.zp_out - c_res) * (1ll << s);
        short_form = add > -(1ll << 31) && add < (1ll << 31);
    }
    if (!short_form) c_res = 0;
    if (res_k8) *res_k8 = short_form ? k8 : 0xFFFFFFFFu;
    for (int o = 0; o < G.coutp; ++o) {
        const int s = shift[o] - 1;
        out4[4 * o + 0] = bias_folded[o];
        out4[4 * o + 1] = mult[o];
        out4[4 * o + 2] = s >= 1 ? (int32_t)((1ll << (s - 1)) + ((long long)G.zp_out - c_res) * (1ll << s)) : 0;
        out4[4 * o + 3] = s >= 1 ? s : 0;
    }
    return fast;
}

cudaError_t launch_igemm_conv(const GLayer &G, const int8_t *wpack, const int32_t *cst, bool fast, uint32_t res_k8, int batch, const int8_t *in,
                              const int8_t *res, int8_t *out, int32_t *err, cudaStream_t st, bool debug_stall, bool tensor_copy)
{
    IgemmParams p;
    p.L = G;
    p.cst = reinterpret_cast<const int4 *>(cst);
    p.fast_requant = fast ? 1 : 0;
    p.lo = G.relu ? (G.zp_out > -128 ? G.zp_out : -128) : -128;
    const int res_n = 31 - G.res_shift;
    p.fast_residual = (res_n == 31 || res_n == 32) ? 1 : 0;
    p.debug_stall = debug_stall ? 1 : 0;
    // A 1 x 1 stride-1 layer reads its input as the matrix [pixel][channel]: the tile's operand rows are a box of the
    // view (16 bytes, pixel, 16-byte column) and come by tensor copy.  The encoder is the driver's, looked up at run
    // time; without it (or if it refuses the view) the gather warps do the work.
    p.tma_a = 0;
    memset(&p.tmap_a, 0, sizeof(p.tmap_a));
    if (tensor_copy && G.kh == 1 && G.kw == 1 && G.stride == 1 && G.pad == 0) {
        typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                     const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
        static EncodeFn encode = nullptr;
        static bool looked_up = false;
        if (!looked_up) {
            void *fn = nullptr;
            cudaDriverEntryPointQueryResult qr;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
                encode = (EncodeFn)fn;
            else
                cudaGetLastError();
            looked_up = true;
        }
        if (encode) {
            const cuuint64_t dims[3] = {16, (cuuint64_t)batch * G.hin * G.win, (cuuint64_t)(G.cinp / 16)};
            const cuuint64_t strides[2] = {(cuuint64_t)G.cinp, 16};
            const cuuint32_t box[3] = {16, (cuuint32_t)kTileM, (cuuint32_t)(kBlockK / 16)}, estr[3] = {1, 1, 1};
            const CUresult r = encode(&p.tmap_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t *>(in), dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r == CUDA_SUCCESS) p.tma_a = 1;
            else if (getenv("ISC_DEBUG_CUDA")) fprintf(stderr, "isc: cuTensorMapEncodeTiled: %d\n", (int)r);
        }
    }
    p.res_m2 = 0; p.res_r2 = 0;
    p.res_short = (res && res_k8 != 0xFFFFFFFFu) ? 1 : 0;
    p.res_k8 = p.res_short ? res_k8 : 0u;
    if (res && p.fast_residual) {
        p.res_m2 = (uint32_t)((unsigned long long)(uint32_t)G.res_mult << (32 - res_n));
        p.res_r2 = ((1ll << (res_n - 1)) - (128ll + G.zp_res) * (long long)G.res_mult) * (1ll << (32 - res_n));
    }
    p.batch = batch;
    p.n_tile = igemm_tile_n(G);
    if (p.n_tile == 0) return cudaErrorInvalidValue;
    p.tmem_cols = 2 * p.n_tile;                                  // two accumulators: 128, 256 or 512 columns
    const long long m_total = (long long)batch * G.hout * G.wout;
    if (m_total >= (1ll << 31) / (G.coutp / p.n_tile) || (long long)batch * G.hin * G.win * G.cinp >= (1ll << 31)) return cudaErrorInvalidValue;
    p.m_total = (uint32_t)m_total;
    p.tiles_m = (p.m_total + kTileM - 1) / kTileM;
    p.in = in; p.res = res; p.out = out; p.wpack = wpack; p.err = err;
    if (p.tiles_m == 0) return cudaSuccess;
    // as many operand stages as fit beside the constants, at most kMaxStages
    const size_t stage_bytes = (size_t)kTileM * kBlockK + (size_t)p.n_tile * kBlockK, cst_bytes = (size_t)G.coutp * 16;
    const size_t scratch_bytes = (size_t)kAllEpiWarps * 32 * ((size_t)p.n_tile / (kEpiWarps / 4) + 16);
    const size_t smem_limit = 226 * 1024;
    if (cst_bytes + scratch_bytes + 2 * stage_bytes > smem_limit) return cudaErrorInvalidValue;
    p.stages = (int)std::min<size_t>(kMaxStages, (smem_limit - cst_bytes - scratch_bytes) / stage_bytes);
    p.scratch_off = (uint32_t)((size_t)p.stages * stage_bytes + cst_bytes);
    const size_t smem = (size_t)p.stages * stage_bytes + cst_bytes + scratch_bytes;
    static int n_sms = 0;
    if (n_sms == 0) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_igemm, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_limit);
        if (e != cudaSuccess) { n_sms = 0; return e; }
    }
    // persistent: one CTA per SM (shared memory and the 512 tensor-memory columns allow no second one at N = 256)
    const uint32_t n_tiles = p.tiles_m * (uint32_t)(G.coutp / p.n_tile);
    const unsigned grid = std::min<uint32_t>(n_tiles, (uint32_t)n_sms);
    k_igemm<<<grid, kGemmThreads, smem, st>>>(p);
    return cudaGetLastError();
}

// ---- the stem

namespace {

int stem_band_rows(const GLayer &G)
{
    const int wpad = G.win + 2 * G.pad + 8;
    int rows = 8;
    while (rows > 1 && (size_t)((rows - 1) * G.stride + G.kh) * wpad * 4 > 24 * 1024) rows >>= 1;
    return rows;
}

}  // namespace

bool stem_fits(const GLayer &G, int in_c)
{
    if (G.op != ISC_CONV2D || in_c > 4 || G.kw > 8 || G.kh > 8 || G.coutp % 16 != 0 || G.coutp > 256) return false;
    const int rows = stem_band_rows(G);
    const size_t patch = (size_t)((rows - 1) * G.stride + G.kh) * (G.win + 2 * G.pad + 8) * 4;
    const size_t total = (size_t)G.kh * G.coutp * 32 + 2 * (size_t)G.kh * kTileM * 32 + patch;
    return total <= 100 * 1024;
}

size_t stem_pack_bytes(const GLayer &G) { return (size_t)G.kh * G.coutp * 32; }

// w: [cout][cin][kh][kw] -> [filter row][2 columns of 16 bytes][coutp rows][16]: byte pix * 4 + ch of a row's 32
void stem_pack_weights(const GLayer &G, const int8_t *w, int8_t *out)
{
    size_t at = 0;
    for (int r = 0; r < G.kh; ++r)
        for (int j = 0; j < 2; ++j)
            for (int n = 0; n < G.coutp; ++n)
                for (int e = 0; e < 16; ++e, ++at) {
                    const int c32 = j * 16 + e, pix = c32 >> 2, ch = c32 & 3;
                    out[at] = (n < G.cout && pix < G.kw && ch < G.cin) ? w[(((size_t)n * G.cin + ch) * G.kh + r) * G.kw + pix] : (int8_t)0;
                }
}

cudaError_t launch_stem_conv(const GLayer &G, const int8_t *wpack, const int32_t *cst, bool fast, const uint8_t *x_chw, int in_c,
                             const NoiseStream &ns, int batch, int8_t *out, int32_t *err, cudaStream_t st)
{
    StemParams p;
    p.L = G;
    p.in_c = in_c;
    p.band_rows = stem_band_rows(G);
    p.n_bands = (G.hout + p.band_rows - 1) / p.band_rows;
    p.tiles_per_band = (p.band_rows * G.wout + kTileM - 1) / kTileM;
    int cols = 32;
    while (cols < 2 * G.coutp) cols <<= 1;
    p.tmem_cols = cols;
    p.w_bytes = (uint32_t)stem_pack_bytes(G);
    p.patch_bytes = (uint32_t)(((p.band_rows - 1) * G.stride + G.kh) * (G.win + 2 * G.pad + 8) * 4);
    p.x = x_chw; p.ns = ns; p.wpack = wpack;
    p.cst = reinterpret_cast<const int4 *>(cst);
    p.fast_requant = fast ? 1 : 0;
    p.lo = G.relu ? (G.zp_out > -128 ? G.zp_out : -128) : -128;
    p.out = out; p.err = err;
    size_t smem = (size_t)p.w_bytes + 2 * (size_t)G.kh * kTileM * 32 + p.patch_bytes;
    // the noise tables go to shared memory when two CTAs per SM still fit and the guide table follows the cumulative one
    const size_t tab_bytes = ((size_t)(2 * ns.T + 1 + kNoiseGuide + 1) * 4 + 15) & ~(size_t)15;
    p.tab_off = 0;
    if (ns.guide == ns.cum + (2 * ns.T + 1) && smem + tab_bytes <= kStemSmemLimit) {
        p.tab_off = (uint32_t)smem;
        smem += tab_bytes;
    }
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_stem, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStemSmemLimit);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    if (batch <= 0) return cudaSuccess;
    dim3 grid((unsigned)p.n_bands, (unsigned)batch);
    k_stem<<<grid, kStemThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace isc

