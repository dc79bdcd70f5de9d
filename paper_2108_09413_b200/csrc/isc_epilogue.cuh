// The integer epilogue of a convolution / FC output in the layer-by-layer kernels: requantisation by fixed-point
// multiplier and shift, residual term, zero-points and clamps, written with 64-bit arithmetic exactly as the layer
// definition in isc.h states it.
#pragma once

#include <stdint.h>

#include "isc_internal.h"

namespace isc {

// rs(acc * mult, 31 + shift) + residual term + zp_out, clamped to int8 (lower clamp `lo`).
__device__ __forceinline__ int requant_clamp(int acc, int mult, int shift, long long res_term, int zp_out, int lo)
{
    const int n = 31 + shift;
    long long v = ((long long)acc * (long long)mult + (1ll << (n - 1))) >> n;
    v += res_term + zp_out;
    v = v < lo ? lo : v;
    v = v > 127 ? 127 : v;
    return (int)v;
}

__device__ __forceinline__ long long residual_term(int r, int zp_res, int res_mult, int res_shift)
{
    const int n = 31 - res_shift;
    return ((long long)(r - zp_res) * (long long)res_mult + (1ll << (n - 1))) >> n;
}

__device__ __forceinline__ int byte_of(uint32_t w, int i) { return (int)(int8_t)((w >> (8 * i)) & 0xFF); }

// 16 accumulators -> 16 int8 outputs (one uint4), with optional residual read.
__device__ __forceinline__ uint4 epilogue16(const int *acc, const GLayer &L, int o0, const int8_t *res_px)
{
    uint32_t packed[4] = {0, 0, 0, 0};
    uint4 rv = make_uint4(0, 0, 0, 0);
    if (res_px) rv = *reinterpret_cast<const uint4 *>(res_px + o0);
    const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
    const int lo = L.relu ? max(-128, L.zp_out) : -128;
#pragma unroll
    for (int o = 0; o < 16; ++o) {
        int q = 0;
        if (o0 + o < L.cout) {
            long long rt = 0;
            if (res_px) rt = residual_term(byte_of(rw[o >> 2], o & 3), L.zp_res, L.res_mult, L.res_shift);
            q = requant_clamp(acc[o], __ldg(L.mult + o0 + o), __ldg(L.shift + o0 + o), rt, L.zp_out, lo);
        }
        packed[o >> 2] |= (uint32_t)(q & 0xFF) << (8 * (o & 3));
    }
    return make_uint4(packed[0], packed[1], packed[2], packed[3]);
}

}  // namespace isc
