// Layer-by-layer engine: one kernel launch per layer over a batch of noisy samples, int8
// activations in global memory as [sample][y][x][channel padded to 16].  It runs every layer
// type of the ABI and any shape; the shared-memory-resident tensor-core engine
// (isc_line.cu) takes over for the CIFAR-shaped residual networks it is specialised for.
//
// The noisy copies of the image (Def. 3.4: x + delta, delta ~ discrete Gaussian of Eq. 2)
// are produced inside the first convolution's input staging and never written to memory.
#include <cuda_runtime.h>
#include <stdint.h>

#include "isc_epilogue.cuh"
#include "isc_internal.h"

namespace isc {

namespace {

// ------------------------------------------------------------------ random stream

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and xors,
// the key advanced by the Weyl constants between rounds.
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

// Smallest table index k in [0, 2T] with u < cum[k]; 2T when there is none.
__device__ __forceinline__ int dgauss_index(uint32_t u, const uint32_t *__restrict__ cum, int T)
{
    int lo = 0, hi = 2 * T;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (u < __ldg(cum + mid)) hi = mid; else lo = mid + 1;
    }
    return lo;
}

__device__ __forceinline__ uint4 sample_counter(const NoiseStream &ns, int64_t j, uint32_t block)
{
    return make_uint4(block, (uint32_t)(j & 0xFFFFFFFFll), ns.ctr2,
                      ns.ctr3_fixed | (uint32_t)(((j >> 32) & 0xFF) << 8));
}

__device__ __forceinline__ uint32_t word_of(const uint4 &v, int i)
{
    return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}

// ------------------------------------------------------------------ dot products

__device__ __forceinline__ int dp4a_ss(int a, int b, int c) { return __dp4a(a, b, c); }

__device__ __forceinline__ int dp4a_us(uint32_t a, int b, int c)
{
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// ------------------------------------------------------------------ first convolution

// One block = one sample x one band of output rows.  The band's input rows are drawn
// (Philox -> table search -> add -> saturate to 0..255) into shared memory as [row][col][4]
// bytes, then every thread computes output pixels x 16 output channels from that patch.
__global__ void __launch_bounds__(128)
k_first_conv(GLayer L, const uint8_t *__restrict__ x, int in_c, NoiseStream ns, int band_rows,
             int8_t *__restrict__ out)
{
    extern __shared__ uint32_t patch[];   // [rows_in][wpad] packed 4 channels
    const int b = blockIdx.y;
    const int64_t j = ns.first_sample + b;
    const int oy0 = blockIdx.x * band_rows;
    const int oy1 = min(L.hout, oy0 + band_rows);
    const int wpad = L.win + 2 * L.pad;
    const int iy0 = oy0 * L.stride - L.pad;                       // first input row of the patch
    const int rows_in = (oy1 - oy0 - 1) * L.stride + L.kh;
    const uint32_t zp_fill = (uint32_t)(L.zp_in & 0xFF) * (0x01010101u >> (8 * (4 - in_c)));   // padding value = zp_in

    for (int i = threadIdx.x; i < rows_in * wpad; i += blockDim.x) patch[i] = zp_fill;
    __syncthreads();

    // valid input rows of this band
    const int vy0 = max(0, iy0), vy1 = min(L.hin, iy0 + rows_in);
    if (vy1 > vy0) {
        uint8_t *pb = reinterpret_cast<uint8_t *>(patch);
        for (int c = 0; c < in_c; ++c) {
            const int64_t e_begin = ((int64_t)c * L.hin + vy0) * L.win;
            const int64_t e_end = ((int64_t)c * L.hin + vy1) * L.win;
            const int64_t q_begin = e_begin >> 2, q_end = (e_end + 3) >> 2;
            for (int64_t q = q_begin + threadIdx.x; q < q_end; q += blockDim.x) {
                const uint4 r = philox4x32_10(sample_counter(ns, j, (uint32_t)q), ns.key0, ns.key1);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int64_t e = q * 4 + k;
                    if (e < e_begin || e >= e_end) continue;
                    const int rem = (int)(e - (int64_t)c * L.hin * L.win);
                    const int h = rem / L.win, w = rem - h * L.win;
                    const int delta = dgauss_index(word_of(r, k), ns.cum, ns.T) - ns.T;
                    int v = (int)__ldg(x + e) + delta;
                    v = min(255, max(0, v));
                    pb[((h - iy0) * wpad + (w + L.pad)) * 4 + c] = (uint8_t)v;
                }
            }
        }
    }
    __syncthreads();

    const int groups = L.coutp >> 4;
    const int items = (oy1 - oy0) * L.wout * groups;
    const int taps = L.kh * L.kw;
    const int32_t *w32 = reinterpret_cast<const int32_t *>(L.w);
    for (int it = threadIdx.x; it < items; it += blockDim.x) {
        const int g = it / ((oy1 - oy0) * L.wout);
        const int p = it - g * ((oy1 - oy0) * L.wout);
        const int oyl = p / L.wout, ox = p - oyl * L.wout;
        int acc[16];
#pragma unroll
        for (int o = 0; o < 16; ++o) acc[o] = __ldg(L.bias + g * 16 + o);
        for (int r = 0; r < L.kh; ++r)
            for (int s = 0; s < L.kw; ++s) {
                const uint32_t a = patch[(oyl * L.stride + r) * wpad + ox * L.stride + s];
                const int32_t *wp = w32 + (size_t)(g * 16) * taps + r * L.kw + s;
#pragma unroll
                for (int o = 0; o < 16; ++o) acc[o] = dp4a_us(a, __ldg(wp + (size_t)o * taps), acc[o]);
            }
        const uint4 v = epilogue16(acc, L, g * 16, nullptr);
        const size_t px = ((size_t)b * L.hout + (oy0 + oyl)) * L.wout + ox;
        *reinterpret_cast<uint4 *>(out + px * L.coutp + g * 16) = v;
    }
}

// Debug aid: the noisy, saturated input of each sample as [sample][C][H][W] int32.
__global__ void k_noisy_input(const uint8_t *__restrict__ x, int d, NoiseStream ns, int batch,
                              int32_t *__restrict__ out)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nq = ((int64_t)d + 3) >> 2;
    if (idx >= nq * batch) return;
    const int b = (int)(idx / nq);
    const int64_t q = idx - (int64_t)b * nq;
    const uint4 r = philox4x32_10(sample_counter(ns, ns.first_sample + b, (uint32_t)q), ns.key0, ns.key1);
    for (int k = 0; k < 4; ++k) {
        const int64_t e = q * 4 + k;
        if (e >= d) break;
        const int delta = dgauss_index(word_of(r, k), ns.cum, ns.T) - ns.T;
        out[(int64_t)b * d + e] = min(255, max(0, (int)x[e] + delta));
    }
}

// ------------------------------------------------------------------ generic convolution / FC

// thread = one output pixel x 16 output channels; int8 x int8 dot products four at a time.
__global__ void __launch_bounds__(128)
k_conv(GLayer L, int batch, const int8_t *__restrict__ in, const int8_t *__restrict__ res,
       int8_t *__restrict__ out)
{
    const int64_t npx = (int64_t)batch * L.hout * L.wout;
    const int64_t px = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (px >= npx) return;
    const int g = blockIdx.y;
    const int ox = (int)(px % L.wout);
    const int oy = (int)((px / L.wout) % L.hout);
    const int b = (int)(px / ((int64_t)L.wout * L.hout));
    const int c16s = L.cinp >> 4;
    const int taps = L.kh * L.kw;
    const uint32_t zp4 = (uint32_t)(L.zp_in & 0xFF) * 0x01010101u;

    int acc[16];
#pragma unroll
    for (int o = 0; o < 16; ++o) acc[o] = __ldg(L.bias + g * 16 + o);

    for (int r = 0; r < L.kh; ++r) {
        const int iy = oy * L.stride + r - L.pad;
        for (int s = 0; s < L.kw; ++s) {
            const int ix = ox * L.stride + s - L.pad;
            const bool inside = iy >= 0 && iy < L.hin && ix >= 0 && ix < L.win;
            const uint4 *ap = reinterpret_cast<const uint4 *>(
                in + (((size_t)b * L.hin + (inside ? iy : 0)) * L.win + (inside ? ix : 0)) * L.cinp);
            const uint4 *wp = reinterpret_cast<const uint4 *>(L.w) +
                              ((size_t)(g * taps + r * L.kw + s) * c16s) * 16;
            for (int c = 0; c < c16s; ++c) {
                const uint4 a = inside ? __ldg(ap + c) : make_uint4(zp4, zp4, zp4, zp4);
#pragma unroll
                for (int o = 0; o < 16; ++o) {
                    const uint4 wv = __ldg(wp + c * 16 + o);
                    int t = acc[o];
                    t = dp4a_ss((int)a.x, (int)wv.x, t);
                    t = dp4a_ss((int)a.y, (int)wv.y, t);
                    t = dp4a_ss((int)a.z, (int)wv.z, t);
                    t = dp4a_ss((int)a.w, (int)wv.w, t);
                    acc[o] = t;
                }
            }
        }
    }
    const int8_t *res_px = res ? res + (size_t)px * L.coutp : nullptr;
    const uint4 v = epilogue16(acc, L, g * 16, res_px);
    *reinterpret_cast<uint4 *>(out + (size_t)px * L.coutp + g * 16) = v;
}

// ------------------------------------------------------------------ pools

__global__ void k_gavgpool(GLayer L, int batch, const int8_t *__restrict__ in, int8_t *__restrict__ out)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= batch * L.cinp) return;
    const int b = idx / L.cinp, c = idx - b * L.cinp;
    int q = 0;
    if (c < L.cin) {
        const int hw = L.hin * L.win;
        long long sum = 0;
        const int8_t *p = in + (size_t)b * hw * L.cinp + c;
        for (int i = 0; i < hw; ++i) sum += (int)p[(size_t)i * L.cinp] - L.zp_in;
        const int n = 31 + __ldg(L.shift);
        long long v = (sum * (long long)__ldg(L.mult) + (1ll << (n - 1))) >> n;
        v += L.zp_out;
        const int lo = L.relu ? max(-128, L.zp_out) : -128;
        v = v < lo ? lo : v;
        v = v > 127 ? 127 : v;
        q = (int)v;
    }
    out[idx] = (int8_t)q;
}

__global__ void k_maxpool(GLayer L, int batch, const int8_t *__restrict__ in, int8_t *__restrict__ out)
{
    const int c16s = L.cinp >> 4;
    const int64_t total = (int64_t)batch * L.hout * L.wout * c16s;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int g = (int)(idx % c16s);
    const int64_t px = idx / c16s;
    const int ox = (int)(px % L.wout);
    const int oy = (int)((px / L.wout) % L.hout);
    const int b = (int)(px / ((int64_t)L.wout * L.hout));
    uint4 m = make_uint4(0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u);
    for (int r = 0; r < L.kh; ++r) {
        const int iy = oy * L.stride + r - L.pad;
        if (iy < 0 || iy >= L.hin) continue;
        for (int s = 0; s < L.kw; ++s) {
            const int ix = ox * L.stride + s - L.pad;
            if (ix < 0 || ix >= L.win) continue;
            const uint4 a = __ldg(reinterpret_cast<const uint4 *>(
                in + (((size_t)b * L.hin + iy) * L.win + ix) * L.cinp) + g);
            m.x = __vmaxs4(m.x, a.x); m.y = __vmaxs4(m.y, a.y);
            m.z = __vmaxs4(m.z, a.z); m.w = __vmaxs4(m.w, a.w);
        }
    }
    *reinterpret_cast<uint4 *>(out + (size_t)px * L.cinp + g * 16) = m;
}

// ------------------------------------------------------------------ votes

// thread = one sample: argmax over the logits (lowest index wins ties), one vote.
// Votes are first gathered per block in shared memory, then added to the global counts.
__global__ void k_votes(const int8_t *__restrict__ logits, int cp, int n_classes, int batch,
                        int32_t *__restrict__ counts, int8_t *__restrict__ logits_out)
{
    extern __shared__ int32_t hist[];
    for (int i = threadIdx.x; i < n_classes; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) {
        const int8_t *p = logits + (size_t)b * cp;
        int best = 0, bestv = p[0];
        for (int k = 1; k < n_classes; ++k) {
            const int v = p[k];
            if (v > bestv) { bestv = v; best = k; }
        }
        atomicAdd(&hist[best], 1);
        if (logits_out)
            for (int k = 0; k < n_classes; ++k) logits_out[(size_t)b * n_classes + k] = p[k];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n_classes; i += blockDim.x)
        if (hist[i]) atomicAdd(counts + i, hist[i]);
}

}  // namespace

// ------------------------------------------------------------------ launchers

cudaError_t launch_first_conv(const GLayer &L, const uint8_t *x_chw, int in_c, const NoiseStream &ns,
                              int batch, int8_t *out, cudaStream_t st)
{
    const int wpad = L.win + 2 * L.pad;
    int band = 8;
    while (band > 1 && (size_t)((band - 1) * L.stride + L.kh) * wpad * 4 > 40 * 1024) band >>= 1;
    const size_t smem = (size_t)((band - 1) * L.stride + L.kh) * wpad * 4;
    if (smem > 48 * 1024) return cudaErrorInvalidValue;
    dim3 grid((L.hout + band - 1) / band, batch);
    k_first_conv<<<grid, 128, smem, st>>>(L, x_chw, in_c, ns, band, out);
    return cudaGetLastError();
}

cudaError_t launch_noisy_input(const uint8_t *x_chw, int in_c, int in_h, int in_w, const NoiseStream &ns,
                               int batch, int32_t *out_chw, cudaStream_t st)
{
    const int d = in_c * in_h * in_w;
    const int64_t n = (((int64_t)d + 3) >> 2) * batch;
    k_noisy_input<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(x_chw, d, ns, batch, out_chw);
    return cudaGetLastError();
}

cudaError_t launch_conv(const GLayer &L, int batch, const int8_t *in, const int8_t *res, int8_t *out,
                        cudaStream_t st)
{
    const int64_t npx = (int64_t)batch * L.hout * L.wout;
    dim3 grid((unsigned)((npx + 127) / 128), L.coutp >> 4);
    k_conv<<<grid, 128, 0, st>>>(L, batch, in, res, out);
    return cudaGetLastError();
}

cudaError_t launch_gavgpool(const GLayer &L, int batch, const int8_t *in, int8_t *out, cudaStream_t st)
{
    const int n = batch * L.cinp;
    k_gavgpool<<<(n + 127) / 128, 128, 0, st>>>(L, batch, in, out);
    return cudaGetLastError();
}

cudaError_t launch_maxpool(const GLayer &L, int batch, const int8_t *in, int8_t *out, cudaStream_t st)
{
    const int64_t n = (int64_t)batch * L.hout * L.wout * (L.cinp >> 4);
    k_maxpool<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(L, batch, in, out);
    return cudaGetLastError();
}

cudaError_t launch_votes(const int8_t *logits_nhwc, int cp, int n_classes, int batch, int32_t *counts,
                         int8_t *logits_out, cudaStream_t st)
{
    k_votes<<<(batch + 127) / 128, 128, n_classes * sizeof(int32_t), st>>>(logits_nhwc, cp, n_classes, batch,
                                                                          counts, logits_out);
    return cudaGetLastError();
}

}  // namespace isc
