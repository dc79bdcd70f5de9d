/*
 * isc.h -- integer smoothing certification on one NVIDIA B200 (sm_100a).
 *
 * C ABI of the Monte-Carlo PREDICT / CERTIFY loop of integer randomized smoothing
 * (Lin, Lou, Xiong, Shahabi, "Integer-arithmetic-only Certified Robustness for
 * Quantized Neural Networks", ICCV 2021).  For one uint8 image the loop draws N copies
 * perturbed with discrete Gaussian noise (Def. 3.3, Eq. 2), evaluates an int8
 * integer-only classifier f on each copy (Def. 3.4, Eq. 3) and counts the argmax
 * labels; the counts give the predicted class and the certified l2 radius
 * (Algorithm 1, Algorithm 2).
 *
 * Every step runs in CUDA kernels of this library; there is no CPU fallback.  All
 * entry points return ISC_OK (0) or a negative isc_status; they never throw or abort,
 * and on error the output arguments are left untouched.  ABSTAIN is not an error: the
 * class is reported as -1 and the radius as 0.
 *
 * Pointers are HOST pointers unless the argument is documented otherwise.  The caller
 * owns everything it passes; the library copies what it keeps.  Calls on one model
 * handle must not overlap in time (the handle owns its device work space); different
 * handles are independent.  `cuda_stream` is a cudaStream_t passed as void* (NULL =
 * the default stream); each call returns after its work on that stream has completed.
 */
#ifndef ISC_H_
#define ISC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ISC_OK = 0,
    ISC_ERR_ARG = -1,          /* null pointer, value out of range                          */
    ISC_ERR_SHAPE = -2,        /* layer list does not type-check (channels, sizes, tensors) */
    ISC_ERR_UNSUPPORTED = -3,  /* valid, but outside what the kernels implement             */
    ISC_ERR_NOMEM = -4,        /* host or device allocation failed                          */
    ISC_ERR_CUDA = -5,         /* a CUDA call or kernel launch failed                       */
    ISC_ERR_TIMEOUT = -6       /* a bounded device-side wait expired; results discarded     */
} isc_status;

typedef enum { ISC_CONV2D = 0, ISC_FC = 1, ISC_GAVGPOOL = 2, ISC_MAXPOOL = 3 } isc_op;

/*
 * One layer of the quantized base classifier f.  Tensor 0 is the (noisy, saturated)
 * uint8 network input; layer i reads tensor `in_tensor` (<= i) and writes tensor i+1;
 * the last tensor holds the n_classes logits.  The paper delegates the layer
 * arithmetic to the integer-only quantization scheme it cites (Sec. 1 and Sec. 2,
 * "Model Compression: Quantization"); this library fixes it as follows, with
 * rs(v, n) = floor(v / 2^n + 1/2) evaluated exactly:
 *
 *   conv / FC : acc[o] = bias[o] + sum_{c,r,s} (a[c, y*stride+r-pad, x*stride+s-pad] - zp_in) * w[o,c,r,s]
 *               (taps outside the image contribute 0), int32 accumulation;
 *               v = rs(acc * mult[o], 31 + shift[o]);
 *               if res_tensor >= 0:  v += rs((r[o,y,x] - zp_res) * res_mult, 31 - res_shift);
 *               out = min(127, max(lo, v + zp_out)),  lo = relu ? max(-128, zp_out) : -128.
 *   global average pool : s = sum over pixels of (a - zp_in); out = clamp(rs(s * mult[0], 31 + shift[0]) + zp_out).
 *   max pool  : integer maximum over the taps inside the image; zero-point unchanged.
 *
 * Ranges: mult in [2^30, 2^31), shift in [0, 31], res_mult in [2^30, 2^31) when a
 * residual is present, res_shift in [-4, 4], zero-points in [-128, 127] (zp_in of a
 * layer reading tensor 0 in [0, 255]).  Weights are symmetric int8 (zero-point 0).
 */
typedef struct {
    int32_t op;                       /* isc_op                                               */
    int32_t in_tensor, res_tensor;    /* res_tensor = -1: no residual add                     */
    int32_t cin, cout, kh, kw, stride, pad; /* FC: 1x1 on a 1x1 map; pools: cout = cin        */
    int32_t relu;                     /* 1: lower clamp is max(-128, zp_out)                  */
    int32_t zp_in, zp_out, zp_res;
    const int8_t *w;                  /* [cout][cin][kh][kw]; NULL for pools                  */
    const int32_t *bias;              /* [cout]; NULL for pools                               */
    const int32_t *mult;              /* [cout]; pools: [1]                                   */
    const int8_t *shift;              /* [cout]; pools: [1]                                   */
    int32_t res_mult, res_shift;
} isc_layer;

typedef struct isc_model isc_model;   /* opaque; owns the device copies of all parameters    */

/*
 * isc_load_qmodel -- validate a layer list, repack it for the GPU and upload it.
 * The base classifier f of Def. 3.4 / Algorithm 1's "base function f".
 *   layers[n_layers] : as above; may be freed on return.
 *   in_c, in_h, in_w : shape of the CHW uint8 network input.
 *   n_classes        : size of the last tensor (must be C x 1 x 1 with C = n_classes).
 *   out              : receives the handle; release it with isc_free_qmodel.
 * Errors: ISC_ERR_ARG, ISC_ERR_SHAPE, ISC_ERR_UNSUPPORTED, ISC_ERR_NOMEM, ISC_ERR_CUDA.
 */
int isc_load_qmodel(const isc_layer *layers, int n_layers, int in_c, int in_h, int in_w,
                    int n_classes, isc_model **out);

void isc_free_qmodel(isc_model *m);

/*
 * isc_plan_resident -- host-only query: would isc_load_qmodel place this network on the
 * shared-memory-resident tensor-core engine (engine 3)?  Validates the layer list exactly as
 * isc_load_qmodel does and runs the engine's planner; touches no GPU.
 *   returns        : 1 = fits, 0 = valid but served by the layer-by-layer kernels, < 0 = isc_status
 *   out_rule       : 0 when it fits, else the number of the planner rule that refused it (NULL to skip)
 *   out_smem_bytes : shared memory per CTA the plan needs when it fits (NULL to skip)
 */
int isc_plan_resident(const isc_layer *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes,
                      int32_t *out_rule, int64_t *out_smem_bytes);

/*
 * isc_predict -- Algorithm 2 (Appendix C): N noisy evaluations, top two vote counts
 * (n_A, n_B), two-sided exact binomial test of n_A out of n_A + n_B at 1/2; the class
 * is returned iff the p-value is <= alpha, else -1 (ABSTAIN).
 *   x_u8       : host, CHW, in_c*in_h*in_w bytes.
 *   seed, image_id : select the random stream (see isc_sample_counts); phase 2 is used.
 *   N >= 1, sigma > 0 (noise std in [0,1] pixel units, i.e. 255*sigma pixel levels),
 *   0 < alpha < 1.
 *   out_class  : host, one int32.   out_counts : host, n_classes int32, or NULL.
 */
int isc_predict(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id,
                int64_t N, double sigma, double alpha, void *cuda_stream,
                int32_t *out_class, int32_t *out_counts);

/*
 * isc_certify -- Algorithm 1: N0 noisy evaluations select the class c_A (phase 0), N
 * fresh ones count its votes n_A (phase 1); p_A is the one-sided (1 - alpha)
 * Clopper-Pearson lower bound of n_A out of N; if p_A > 1/2 the result is c_A with
 * radius sigma * Phi^-1(p_A), Phi the standard normal cdf, else ABSTAIN (-1, 0.0).
 * The radius is in the same units as sigma.
 *   out_counts0 / out_counts : host, n_classes int32 each (votes of the two phases), or NULL.
 */
int isc_certify(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id,
                int64_t N0, int64_t N, double sigma, double alpha, void *cuda_stream,
                int32_t *out_class, double *out_radius,
                int32_t *out_counts0, int32_t *out_counts);

/*
 * isc_certify_batch -- Algorithm 1 for n_images images; image i uses image_id0 + i and
 * gives exactly what isc_certify gives for it.
 *   x_u8        : [n_images][C][H][W] bytes; a HOST pointer, or a DEVICE pointer when
 *                 x_on_device != 0 (the images are then read in place).
 *   out_class[n_images], out_radius[n_images] : host.
 *   out_counts0 / out_counts : host, [n_images][n_classes] int32, or NULL.
 */
int isc_certify_batch(isc_model *m, const uint8_t *x_u8, int x_on_device, int n_images,
                      uint64_t seed, uint64_t image_id0, int64_t N0, int64_t N,
                      double sigma, double alpha, void *cuda_stream,
                      int32_t *out_class, double *out_radius,
                      int32_t *out_counts0, int32_t *out_counts);

/*
 * isc_sample_counts -- the Monte-Carlo loop alone (Algorithm 1 steps 1-4, Algorithm 2
 * steps 1-2) for samples j = first_sample .. first_sample + n_samples - 1 of one image:
 * draw delta_j, evaluate f(clamp(x + delta_j, 0, 255)), count the argmax label (ties go
 * to the lowest class index).  Counts over a range equal the sum of the counts over any
 * partition of it, whatever the launch batch.
 * Random stream: element e = (c*H + h)*W + w of sample j takes output word (e & 3) of
 * Philox4x32-10 with key (seed low, seed high) and counter
 *   (e >> 2, j low 32, image_id low 32, phase | (j >> 32 & 0xFF) << 8 | (image_id >> 32 & 0xFFFF) << 16),
 * and maps that uniform u to the smallest level z with u < cum[z], where cum is the
 * 2^-32-grid CDF of Eq. 2 on the integer pixel levels with std 255*sigma, cut at
 * +-ceil(7*255*sigma).  Requires j < 2^40, image_id < 2^48, 0 <= phase < 256.
 *   out_counts : host, n_classes int32 (overwritten).
 *   out_logits : host, [n_samples][n_classes] int8, or NULL.
 */
int isc_sample_counts(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id,
                      int32_t phase, int64_t first_sample, int64_t n_samples, double sigma,
                      void *cuda_stream, int32_t *out_counts, int8_t *out_logits);

/*
 * isc_sample_counts_static -- isc_sample_counts for callers that must not allocate device
 * memory.  (The paper has no counterpart: this is a deployment variant of the same
 * Monte-Carlo loop, added for such callers.)
 *
 * Some hosts of this library may not call cudaMalloc at all once they are running: a
 * service whose device memory is handed out up front by its own pool, a real-time loop
 * that cannot afford the implicit device synchronisation of an allocation, a process
 * running under a memory budget enforced by refusing allocations.  For them this entry
 * point computes the same vote counts as isc_sample_counts with the layer-by-layer
 * kernels, but takes every byte of its device work space (activation buffers, noise
 * table, staged image, counts) from one fixed 32 MiB array that is part of the library
 * image.  It calls no cudaMalloc / cudaFree and no allocating library routine; the model
 * handle must have been loaded beforehand (loading does allocate).  Each GPU on which the
 * library is loaded holds that array until the process exits.
 *
 *   arguments  : as isc_sample_counts (x_u8 and out_counts are host pointers); no logits.
 *   limits     : returns ISC_ERR_UNSUPPORTED, doing nothing, when one sample's activation
 *                buffers do not fit in the array, when the image exceeds 1 MiB, when the
 *                noise table exceeds 16384 entries (sigma above about 4.5) or when
 *                n_classes exceeds 4096.  Any n_samples is accepted: samples are processed
 *                in batches as large as the array allows.
 *   first call : the first call made on a device looks up the array's device address (the
 *                device must be current); make that call before starting a stream capture.
 *   sharing    : all calls, on all handles and streams, share the one array.  Its contents
 *                persist between calls (the counts are cleared at the start of each call);
 *                two calls whose GPU work overlaps in time race on it, so serialise them.
 */
int isc_sample_counts_static(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id,
                             int32_t phase, int64_t first_sample, int64_t n_samples, double sigma,
                             void *cuda_stream, int32_t *out_counts);

/*
 * isc_decide_certify / isc_decide_predict -- the host part of Algorithm 1 (steps 2,
 * 5-9) and Algorithm 2 (steps 2-6) on given vote counts; no GPU work.
 *   out_p_lower : the lower confidence bound p_A, or NULL.
 */
int isc_decide_certify(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N,
                       double sigma, double alpha, int32_t *out_class, double *out_radius,
                       double *out_p_lower);
int isc_decide_predict(const int32_t *counts, int n_classes, double alpha, int32_t *out_class);

/*
 * isc_noise_table -- the cumulative table of the noise law (Eq. 2) the kernels use for
 * `sigma`: writes 2*T+1 uint32 entries for levels -T..T to `cum` (host) when
 * capacity >= 2*T+1, and T to *out_T.  Pass cum = NULL to query T only.
 */
int isc_noise_table(double sigma, uint32_t *cum, int64_t capacity, int32_t *out_T);

/*
 * isc_noise_table_rounded -- the same table for the noise of the paper's comparison method
 * "FloatRS-quant" (Sec. 4.1, comparison methods: continuous Gaussian noise is added to the image
 * and the sum is quantised): on integer pixels delta = round(255 sigma g), g ~ N(0, 1), so
 * cum[z + T] = floor(2^32 * Phi((z + 1/2) / (255 sigma))).  A model handle draws from this law
 * instead of Eq. 2 after isc_set_option(m, "noise", 1); nothing else changes (same random
 * stream, same inverse-CDF rule, same kernels).  Arguments as isc_noise_table.
 */
int isc_noise_table_rounded(double sigma, uint32_t *cum, int64_t capacity, int32_t *out_T);

/*
 * isc_radius_integer -- the integer-only form of the radius (Theorem 3.2 steps 2-3,
 * Theorem 3.1): the quantile of the one-dimensional discrete Gaussian N_Z(0, (255 sigma)^2)
 * by lookup in the cumulative table above, for a probability given as a 32-bit fixed-point
 * fraction p_fx = floor(p * 2^32).  No GPU work, no floating point after the table is built.
 *   out_q         : the smallest pixel level q in [-T, T] with cum[q + T] >= p_fx (T if none);
 *                   q / 255 is the radius in [0,1] pixel units, q <= 0 certifies nothing.
 *   out_q_squared : q * q, the squared integer radius the theorem compares distances with
 *                   (NULL to skip).
 * Returns ISC_ERR_ARG for a bad sigma or a NULL out_q; outputs untouched on error.
 */
int isc_radius_integer(double sigma, uint32_t p_fx, int32_t *out_q, int64_t *out_q_squared);

/*
 * isc_certify_integer / isc_decide_certify_integer -- Algorithm 1 with the radius in the
 * integer form of Theorem 3.2 (steps 2-3): class selection, vote count and the confidence
 * bound p_A are Algorithm 1's (steps 1-6); the radius is then read off the cumulative table
 * of the one-dimensional discrete Gaussian N_Z(0, (255 sigma)^2) (isc_noise_table) at
 * floor(p_A * 2^32) instead of the normal quantile.
 *   two_sided = 0 : out_q = Phi^-1_{N_H}(p_A) in pixel levels (q / 255 is the radius in the
 *                   units of sigma), out_q_squared = q^2, the squared l2 radius the theorem
 *                   compares integer perturbations with.
 *   two_sided = 1 : Theorem 3.1's radius (sigma / 2)(Phi^-1(p_A^lb) - Phi^-1(p_B^ub)), with
 *                   p_B^ub the one-sided (1 - alpha) Clopper-Pearson upper bound of the
 *                   runner-up's votes: out_q = q_A - q_B (TWICE the radius, so that it stays an
 *                   integer), out_q_squared = (q_A - q_B)^2 (four times the squared radius).
 *                   Each bound holds with probability 1 - alpha on its own.
 * ABSTAIN (class -1, q = 0) when p_A <= 1/2, or two-sided when p_A^lb < p_B^ub.
 * isc_decide_certify_integer does the host part on given counts (no GPU work); arguments as
 * isc_decide_certify.  out_q_squared, out_counts0, out_counts may be NULL.
 */
int isc_certify_integer(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id,
                        int64_t N0, int64_t N, double sigma, double alpha, int two_sided,
                        void *cuda_stream, int32_t *out_class, int32_t *out_q, int64_t *out_q_squared,
                        int32_t *out_counts0, int32_t *out_counts);
int isc_decide_certify_integer(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N,
                               double sigma, double alpha, int two_sided, int32_t *out_class,
                               int32_t *out_q, int64_t *out_q_squared);

/*
 * isc_certified_metrics -- Certified Percentage and Certified Accuracy over a set of
 * certification results (Sec. 4.1, Evaluation Metrics, the two displayed equations); host only.
 *   classes, radii : what isc_certify returned for n inputs (class -1 = ABSTAIN), host arrays [n]
 *   labels         : ground-truth classes [n]
 *   r, n_r         : radius thresholds [n_r] (n_r may be 0)
 *   out_cp         : inputs that did not abstain / n (0 for n = 0)
 *   out_ca         : [n_r]; for each threshold, inputs that did not abstain, were classified
 *                    correctly and have radius >= r, divided by the inputs that did not abstain
 *                    (the denominator the equation prints; 0 when none certified)
 * Returns ISC_ERR_ARG for NULL arrays with n > 0, negative sizes or a NULL out_cp.
 */
int isc_certified_metrics(const int32_t *classes, const double *radii, const int32_t *labels, int64_t n,
                          const double *r, int n_r, double *out_cp, double *out_ca);

/*
 * isc_debug_tensor -- evaluate sample j of one image and copy tensor `tensor`
 * (0 = the noisy input, values 0..255; i+1 = output of layer i) to `out` as
 * [C][H][W] int32 (host).  For layer-by-layer comparison; slow.
 */
int isc_debug_tensor(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id,
                     int32_t phase, int64_t j, double sigma, int tensor, void *cuda_stream,
                     int32_t *out, int64_t capacity);

/*
 * isc_debug_wait_timeout -- exercises the bounded-wait failure path of the resident engine
 * without any failure: a one-thread kernel runs the engine's own wait code on a barrier and a
 * counter that nothing ever completes, with `limit_ns` (1,000 .. 100,000,000) as the limit.
 * The GPU keeps running; nothing faults or hangs.
 *   returns : ISC_ERR_TIMEOUT when the path works as designed (the expired wait raised the
 *             engine's error word, and reading it reported and cleared it); ISC_OK means the
 *             wait did NOT expire; ISC_ERR_UNSUPPORTED if the model has no resident engine.
 *   out4    : host, 4 int32: result of the first wait (0 = expired), result of the second wait
 *             (0 = fell through because the abort flag was up), the abort flag, nanoseconds spent.
 * A model without the resident engine but with tensor-core layers (the layer-by-layer tensor-core
 * engine) is probed through that engine instead: one launch of its first implicit-GEMM layer on one
 * sample's work space with the weights held back, so that the kernel's own waits run out (after
 * their fixed limit of two seconds; `limit_ns` is not used) and every role leaves through the abort
 * path.  out4 = {0, 0, the kernel's error word (non-zero = 1 + the CTA that raised it), host
 * nanoseconds of the launch, saturated}.
 * The handle stays usable: the next call on it must succeed.
 */
int isc_debug_wait_timeout(isc_model *m, int64_t limit_ns, void *cuda_stream, int32_t *out4);

/*
 * isc_debug_residual_form -- host only.  The tensor-core engines compute the residual operand's
 * rescale rs((r - zp_res) * res_mult, 31 - res_shift) (the skip path's term of the residual add)
 * as floor((u * m2 + R2) / 2^32), u = r + 128, and, where an offset k < 4096 exists for which
 * floor((256 k + u) * m2 / 2^32) - c equals that for all 256 values of u, in this shorter form.
 * This call runs the search the engines run.
 *   returns : 1 and *k / *c when the form exists, 0 when the engines keep the long form
 *             (including res_shift other than 0 or -1), ISC_ERR_ARG for a null pointer.
 */
int isc_debug_residual_form(int32_t res_mult, int32_t res_shift, int32_t zp_res, int32_t *k, int32_t *c);

/*
 * isc_set_option -- "batch" and "engine" are tuning knobs that change no result; "noise" selects
 * the noise law and therefore changes the samples.
 *   "tensor_copy" : 1 (default) = the layer-by-layer tensor-core engine brings the operand rows of
 *              1 x 1 stride-1 convolutions by tensor copy, 0 = by the copies every other layer uses;
 *              changes no result.
 *   "noise"  : 0 = the discrete Gaussian of Def. 3.3 / Eq. 2 (IntRS, the default), 1 = the
 *              rounded continuous Gaussian of the comparison method (isc_noise_table_rounded).
 *   "batch"  : noisy samples per launch (0 = choose automatically).
 *   "engine" : 0 = automatic (3 if the model fits it, else 2 if any layer fits it, else 1),
 *              1 = layer-by-layer kernels without tensor cores, 2 = layer-by-layer with
 *              the tcgen05 implicit-GEMM kernel for every convolution whose input and
 *              output channels are multiples of 64, 3 = the line-tiled
 *              shared-memory-resident tensor-core kernel (2 and 3 give
 *              ISC_ERR_UNSUPPORTED at the next call if the model does not fit).
 * isc_get_info reads back: "engine" (the engine the last call used), "gpu_launches"
 * (kernel launches issued by this handle so far), "macs_per_sample",
 * "has_line_engine" (1 if the model fits engine 3), "has_tensor_core_layers" (1 if
 * engine 2 has a layer to run) and, for engine 3, "cycles_fill",
 * "cycles_noise", "cycles_conv", "cycles_tail": SM cycles summed over thread blocks and over
 * all launches of this handle so far, spent in halo fills, in the noise phase (draw, add,
 * saturate, store), in the convolutions and in pool / FC / argmax / vote -- the noise
 * sampler's cost share is cycles_noise over their sum (these reads synchronise the device).
 */
int isc_set_option(isc_model *m, const char *name, int64_t value);
int isc_get_info(isc_model *m, const char *name, int64_t *out);

const char *isc_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* ISC_H_ */
