// Microbenchmark: what one thread pays to issue chains of tcgen05.mma (kind::i8, M = 128, N = 48, K = 32), with and
// without the instructions that surround a chain in the line-tiled engine (a dependency test by an acquiring load
// from shared memory, tcgen05.fence::after_thread_sync, tcgen05.commit on every second chain), for a lone lane and
// for a converged warp with an elected lane, with the per-chain values in shared memory or in kernel parameters.
//
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o mma_issue_probe mma_issue_probe.cu && ./mma_issue_probe
//
// Every operand range is checked on the host against the shared-memory allocation before the launch, and the
// completion wait is bounded.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long gtimer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__host__ __device__ inline uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred = 0;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\t@p mov.u32 %0, 1;\n\t}" : "+r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void mma(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc) : "memory");
}
__device__ __forceinline__ void commit_if(uint32_t base, uint32_t off)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0xFFFF;\n\t"
                 "@p tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
                 ::"r"(base + off), "r"(off) : "memory");
}
__device__ __forceinline__ uint32_t ld_acq(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}

constexpr int kOps = 32, kSmem = 96 * 1024, kAOff = 1024, kBOff = 80 * 1024, kPitch16 = 132, kALines = 30;
struct Rec { uint32_t d_col, idesc, a_add, b_add, w0, c0, pad0, pad1; };
struct Params { Rec rec[kOps]; };

// V: 1 lone lane, 2 converged warp with records in shared memory, 3 converged warp with records in kernel parameters
// F: bit 0 acquiring load, bit 1 fence, bit 2 commit, bit 3 one MMA per chain instead of two
template <int V, int F>
__global__ void __launch_bounds__(64) probe(const __grid_constant__ Params P, int reps, long long *out, int *err)
{
    extern __shared__ __align__(1024) uint8_t sm[];
    __shared__ __align__(16) Rec srec[kOps + 1];
    __shared__ __align__(8) unsigned long long bars[kOps];
    __shared__ uint32_t stored[8];
    __shared__ uint32_t tmem_base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < kSmem / 4; i += blockDim.x) ((uint32_t *)sm)[i] = 0x01010101u;
    for (int i = threadIdx.x; i <= kOps; i += blockDim.x) srec[i] = P.rec[i < kOps ? i : 0];
    if (threadIdx.x < kOps) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[threadIdx.x])) : "memory");
    if (threadIdx.x < 8) stored[threadIdx.x] = 0x7FFFFFFF;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base;
    if (warp == 0) {
        const uint32_t ahi = (uint32_t)(make_desc(0, 0, 128) >> 32), bhi = (uint32_t)(make_desc(0, 128, 256) >> 32);
        const uint32_t alo0 = (uint32_t)make_desc(smem_u32(sm) + kAOff, 64, 128), alo1 = (uint32_t)make_desc(smem_u32(sm) + kAOff + 128, 64, 128);
        const uint32_t blo0 = (uint32_t)make_desc(smem_u32(sm) + kBOff, 128, 256), blo1 = (uint32_t)make_desc(smem_u32(sm) + kBOff + 4096, 128, 256);
        const uint32_t full = smem_u32(bars), st = smem_u32(stored);
        long long t0 = 0, t1 = 0;
        if (V == 1) {
            if (lane == 0) {
                t0 = clock64();
                for (int r = 0; r < reps; ++r) {
#pragma unroll 1
                    for (int i = 0; i < kOps; ++i) {
                        const Rec q = srec[i];
                        if (F & 1) { if ((int)(ld_acq(st + q.w0) - 100u) < 0) *err = 2; }
                        if (F & 2) asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t d = tmem + q.d_col;
                        mma(d, ((uint64_t)ahi << 32) | (alo0 + q.a_add), ((uint64_t)bhi << 32) | (blo0 + q.b_add), q.idesc);
                        if (!(F & 8)) mma(d, ((uint64_t)ahi << 32) | (alo1 + q.a_add), ((uint64_t)bhi << 32) | (blo1 + q.b_add), q.idesc);
                        if (F & 4) commit_if(full, q.c0);
                    }
                }
                t1 = clock64();
            }
        } else {
            t0 = clock64();
            for (int r = 0; r < reps; ++r) {
#pragma unroll 1
                for (int i = 0; i < kOps; ++i) {
                    uint32_t d_col, idesc, a_add, b_add, w0, c0;
                    if (V == 2) {
                        const Rec q = srec[i];
                        d_col = q.d_col; idesc = q.idesc; a_add = q.a_add; b_add = q.b_add; w0 = q.w0; c0 = q.c0;
                    } else {
                        d_col = P.rec[i].d_col; idesc = P.rec[i].idesc; a_add = P.rec[i].a_add; b_add = P.rec[i].b_add;
                        w0 = P.rec[i].w0; c0 = P.rec[i].c0;
                    }
                    if (F & 1) { if ((int)(ld_acq(st + w0) - 100u) < 0) *err = 2; }
                    if (F & 2) asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t d = tmem + d_col;
                    if (elect_one()) {
                        mma(d, ((uint64_t)ahi << 32) | (alo0 + a_add), ((uint64_t)bhi << 32) | (blo0 + b_add), idesc);
                        if (!(F & 8)) mma(d, ((uint64_t)ahi << 32) | (alo1 + a_add), ((uint64_t)bhi << 32) | (blo1 + b_add), idesc);
                        if (F & 4) commit_if(full, c0);
                    }
                    __syncwarp();
                }
            }
            t1 = clock64();
        }
        if (lane == 0) {
            // barrier kOps - 1 is not among the records' commits: its single arrival follows everything issued above
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(full + 8 * (kOps - 1)) : "memory");
            const unsigned long long g0 = gtimer();
            bool ok = true;
            while (!mbar_test(full + 8 * (kOps - 1), 0))
                if (gtimer() - g0 > 1000000000ull) { ok = false; break; }
            if (!ok) *err = 1;
            out[0] = t1 - t0;
            out[1] = clock64() - t0;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

static bool in_bounds(const Params &P)
{
    for (int i = 0; i < kOps; ++i) {
        const long a_end = kAOff + 128 + (long)P.rec[i].a_add * 16 + 64 + 128 * 16;     // second K-step, second half, 128 rows
        const long b_end = kBOff + 4096 + (long)P.rec[i].b_add * 16 + (48 / 8 - 1) * 256 + 128 + 128;
        if (a_end > kBOff || b_end > kSmem || P.rec[i].d_col + 48 > 512 || P.rec[i].w0 >= 32) return false;
        if (P.rec[i].c0 != 0xFFFFu && P.rec[i].c0 >= 8u * (kOps - 1)) return false;
    }
    return true;
}

int main()
{
    Params P;
    for (int i = 0; i < kOps; ++i) {
        P.rec[i].d_col = (uint32_t)(16 * (i % 29));
        P.rec[i].idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((48u >> 3) << 17) | ((128u >> 4) << 24);
        P.rec[i].a_add = (uint32_t)(kPitch16 * (i % kALines));
        P.rec[i].b_add = 0;
        P.rec[i].w0 = 4u * (uint32_t)(i % 8);
        P.rec[i].c0 = (i & 1) && i < kOps - 1 ? 8u * (uint32_t)(i / 2) : 0xFFFFu;
        P.rec[i].pad0 = P.rec[i].pad1 = 0;
    }
    if (!in_bounds(P)) { printf("operand ranges out of bounds\n"); return 1; }
    long long *dout;
    int *derr;
    cudaMalloc(&dout, 16);
    cudaMalloc(&derr, 4);
    cudaMemset(derr, 0, 4);
    const int reps = 50;
    bool failed = false;
    auto run = [&](auto kern, const char *name) {
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        kern<<<1, 64, kSmem>>>(P, reps, dout, derr);
        const cudaError_t e = cudaDeviceSynchronize();
        long long h[2] = {0, 0};
        int herr = 0;
        cudaMemcpy(h, dout, 16, cudaMemcpyDeviceToHost);
        cudaMemcpy(&herr, derr, 4, cudaMemcpyDeviceToHost);
        printf("%-52s %6.1f cycles per chain to issue, %6.1f until complete [%s, err=%d]\n", name, (double)h[0] / (reps * kOps),
               (double)h[1] / (reps * kOps), cudaGetErrorString(e), herr);
        cudaMemset(derr, 0, 4);
        if (e != cudaSuccess || herr) failed = true;
    };
    run(probe<1, 7>, "lone lane: acquire + fence + commit");
    if (!failed) run(probe<2, 7>, "converged warp: acquire + fence + commit");
    if (!failed) run(probe<2, 6>, "converged warp: fence + commit");
    if (!failed) run(probe<2, 5>, "converged warp: acquire + commit");
    if (!failed) run(probe<2, 3>, "converged warp: acquire + fence");
    if (!failed) run(probe<2, 0>, "converged warp: two MMAs only");
    if (!failed) run(probe<2, 8>, "converged warp: one MMA only");
    if (!failed) run(probe<3, 0>, "converged warp, kernel parameters: two MMAs only");
    return failed ? 1 : 0;
}
