// Microbenchmark: cycles per back-to-back tcgen05.mma kind::i8 (M = 128, K = 32, K-major no-swizzle operands in
// shared memory) as a function of N, issued by one thread with all descriptors precomputed in registers.
// It gives the tensor-pipe floor that bounds the resident engine's small-N convolutions.
//
//   nvcc -gencode arch=compute_100a,code=sm_100a -O2 -o mma_rate_probe mma_rate_probe.cu && ./mma_rate_probe
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

constexpr int kSmem = 200 * 1024, kAOff = 1024, kBOff = 128 * 1024, kATiles = 8;

__global__ void __launch_bounds__(160) rate(int N, int n_acc, int iters, long long *out, int *err)
{
    extern __shared__ __align__(1024) uint8_t sm[];
    __shared__ __align__(8) unsigned long long full;
    __shared__ uint32_t tmem_base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < kSmem / 4; i += blockDim.x) ((uint32_t *)sm)[i] = 0x01010101u * (i & 3);
    if (threadIdx.x == 0) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&full)) : "memory");
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base;
    if (warp == 4 && lane == 0) {
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((128u >> 4) << 24);
        const uint64_t bd = make_desc(smem_u32(sm) + kBOff, 128, 256);
        uint64_t ad[kATiles];
        uint32_t dd[kATiles];
        for (int k = 0; k < kATiles; ++k) {
            ad[k] = make_desc(smem_u32(sm) + kAOff + (uint32_t)k * 2048u, 16, 128);
            dd[k] = tmem + (uint32_t)(k % n_acc) * (512u / (uint32_t)n_acc);
        }
        const long long t0 = clock64();
        for (int it = 0; it < iters; it += kATiles) {
#pragma unroll
            for (int k = 0; k < kATiles; ++k)
                asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                             ::"r"(dd[k]), "l"(ad[k]), "l"(bd), "r"(idesc) : "memory");
        }
        const long long t1 = clock64();
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&full)) : "memory");
        const unsigned long long g0 = gtimer();
        bool ok = true;
        while (!mbar_test(smem_u32(&full), 0))
            if (gtimer() - g0 > 2000000000ull) { ok = false; break; }
        out[0] = t1 - t0;
        out[1] = clock64() - t0;
        if (!ok) *err = 1;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 4) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

static bool in_bounds(int N, int n_acc)
{
    const long a_end = kAOff + (long)(kATiles - 1) * 2048 + 15 * 128 + 7 * 16 + 16 + 16;   // last byte of the last A tile
    const long b_end = kBOff + (long)(N / 8 - 1) * 256 + 128 + 7 * 16 + 16;
    return a_end <= kBOff && b_end <= kSmem && N % 16 == 0 && N >= 16 && N <= 256 && 512 % n_acc == 0 && N <= 512 / n_acc;
}

int main()
{
    long long *dout;
    int *derr;
    cudaMalloc(&dout, 16);
    cudaMalloc(&derr, 4);
    cudaMemset(derr, 0, 4);
    cudaFuncSetAttribute(rate, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    const int iters = 4000;
    const int cases[][2] = {{16, 8}, {16, 1}, {32, 8}, {48, 8}, {64, 8}, {96, 4}, {128, 4}, {192, 2}, {256, 2}};
    printf("tcgen05.mma kind::i8 M=128 K=32, %d back-to-back instructions from one thread\n", iters);
    for (const auto &c : cases) {
        if (!in_bounds(c[0], c[1])) { printf("N=%d skipped (bounds)\n", c[0]); continue; }
        rate<<<1, 160, kSmem>>>(c[0], c[1], iters, dout, derr);
        const cudaError_t e = cudaDeviceSynchronize();
        long long h[2];
        int herr;
        cudaMemcpy(h, dout, 16, cudaMemcpyDeviceToHost);
        cudaMemcpy(&herr, derr, 4, cudaMemcpyDeviceToHost);
        const double cyc = (double)h[1] / iters;
        printf("N=%3d accumulators=%d: %.1f cycles/MMA  -> %.0f MAC/clk/SM (%.0f%% of 8192)  [%s, timeout=%d]\n", c[0], c[1], cyc,
               128.0 * c[0] * 32 / cyc, 100.0 * 128.0 * c[0] * 32 / cyc / 8192.0, cudaGetErrorString(e), herr);
        if (e != cudaSuccess || herr) return 1;
    }
    return 0;
}
