// Internal declarations shared by the host API and the kernel files of libisc.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "isc.h"

namespace isc {

struct TShape {
    int c, h, w;
    int cp;  // channels padded to a multiple of 16 (device NHWC layout)
};

constexpr int kNoiseGuideBits = 10, kNoiseGuide = 1 << kNoiseGuideBits;

// Where the random stream of one launch starts (Philox4x32-10 key and fixed counter words).
struct NoiseStream {
    uint32_t key0, key1;      // seed halves
    uint32_t ctr2;            // image_id low 32
    uint32_t ctr3_fixed;      // phase | (image_id >> 32 & 0xFFFF) << 16
    int64_t first_sample;     // sample id of batch slot 0
    const uint32_t *cum;      // device, 2T+1 entries
    int T;
    // Optional guide table (device, kNoiseGuide + 1 entries, or null): guide[j] is the search result for the
    // uniform j << (32 - kNoiseGuideBits), a lower bound of the result for every uniform with these top bits.
    const uint32_t *guide;
    int guide_steps;          // bisection steps that close the widest interval [guide[j], guide[j+1]]
};

// One layer as the layer-by-layer kernels see it (device pointers).
struct GLayer {
    int op;
    int cin, cinp, cout, coutp;
    int kh, kw, stride, pad, relu;
    int zp_in, zp_out, zp_res, res_mult, res_shift;
    int hin, win, hout, wout;
    const int8_t *w;        // conv/FC: [coutp/16][kh*kw][cinp/16][16 out][16 in]; first layer: [coutp][kh*kw][4]
    const int32_t *bias;    // [coutp], folded: bias - zp_in * sum(w)
    const int32_t *mult;    // [coutp]
    const int32_t *shift;   // [coutp]
};

// One validated layer with its host arrays, as the engines' planners receive it.
struct LayerIn {
    isc_layer d;
    const int8_t *w;
    const int32_t *bias;
    const int32_t *mult;
    const int8_t *shift;
};

// ---- layer-by-layer engine (isc_generic.cu) ----
cudaError_t launch_first_conv(const GLayer &L, const uint8_t *x_chw, int in_c, const NoiseStream &ns,
                              int batch, int8_t *out, cudaStream_t st);
cudaError_t launch_noisy_input(const uint8_t *x_chw, int in_c, int in_h, int in_w, const NoiseStream &ns,
                               int batch, int32_t *out_chw, cudaStream_t st);
cudaError_t launch_conv(const GLayer &L, int batch, const int8_t *in, const int8_t *res, int8_t *out,
                        cudaStream_t st);
cudaError_t launch_gavgpool(const GLayer &L, int batch, const int8_t *in, int8_t *out, cudaStream_t st);
cudaError_t launch_maxpool(const GLayer &L, int batch, const int8_t *in, int8_t *out, cudaStream_t st);
cudaError_t launch_votes(const int8_t *logits_nhwc, int cp, int n_classes, int batch, int32_t *counts,
                         int8_t *logits_out, cudaStream_t st);

// ---- layer-by-layer tensor-core convolutions (isc_igemm.cu) ----
// Output-channel tile of the implicit-GEMM kernel for this layer (64, 128 or 256), or 0 when the layer does not fit
// it (input channels not a multiple of 64, output channels not a multiple of 64, pools).
int igemm_tile_n(const GLayer &G);
size_t igemm_pack_bytes(const GLayer &G);
void igemm_pack_weights(const GLayer &G, const int8_t *w_oihw, int8_t *out);
// The residual term F(u) = floor((u * m2 + R2) / 2^32), u = r + 128 in 0..255, of the 32-bit epilogues as
// hi32((256 k + u) * m2) - c: the smallest k < 4096 for which the two agree on all 256 inputs (*k8 = 256 k), or false.
bool residual_short_form(int res_mult, int res_shift, int zp_res, uint32_t *k8, int32_t *c);
// Per-channel requantisation constants of the kernel's 32-bit epilogue (4 x int32 per padded output channel); returns
// whether the layer qualifies for it (every shift >= 2).
bool igemm_constants(const GLayer &G, const int32_t *bias_folded, const int32_t *mult, const int32_t *shift, int32_t *out4,
                     bool has_residual, uint32_t *res_k8);
// `cst` / `fast`: what igemm_constants produced (device copy).  `err` (device) receives a non-zero word if a bounded
// wait inside the kernel expired.  `debug_stall`: the kernel's weights are never sent, so that its waits run out
// (after their 2 s limit) and the CTAs leave through the abort path -- nothing faults or hangs.  `tensor_copy`: a
// 1 x 1 stride-1 layer may take its operand rows by tensor copy (false: the gather warps bring them, as for every
// other layer).
cudaError_t launch_igemm_conv(const GLayer &G, const int8_t *wpack, const int32_t *cst, bool fast, uint32_t res_k8, int batch, const int8_t *in,
                              const int8_t *res, int8_t *out, int32_t *err, cudaStream_t st, bool debug_stall = false,
                              bool tensor_copy = true);

// The first convolution (<= 4 input channels, filter at most 8 x 8) on the tensor cores, noise drawn into its staging.
bool stem_fits(const GLayer &G, int in_c);
size_t stem_pack_bytes(const GLayer &G);
void stem_pack_weights(const GLayer &G, const int8_t *w_oihw, int8_t *out);
cudaError_t launch_stem_conv(const GLayer &G, const int8_t *wpack, const int32_t *cst, bool fast, const uint8_t *x_chw, int in_c,
                             const NoiseStream &ns, int batch, int8_t *out, int32_t *err, cudaStream_t st);

// ---- host decision rules (isc_decide.cpp) ----
double lower_conf_bound(int64_t k, int64_t n, double alpha);
double normal_quantile(double p);
double binom_pvalue_half(int64_t n_a, int64_t m);
int32_t decide_certify(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N,
                       double sigma, double alpha, double *radius, double *p_lower);
int32_t decide_predict(const int32_t *counts, int n_classes, double alpha);
int32_t decide_certify_integer(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N, double sigma,
                               double alpha, bool two_sided, int32_t *q, int64_t *q_squared);
int noise_halfwidth(double sigma);
void noise_table(double sigma, std::vector<uint32_t> &cum);
void noise_table_rounded(double sigma, std::vector<uint32_t> &cum);

}  // namespace isc
