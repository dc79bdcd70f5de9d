// Line-tiled shared-memory-resident tensor-core engine for CIFAR-shaped residual networks.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "isc.h"
#include "isc_internal.h"

namespace isc {

struct LinePlan;

// Builds the plan when the network fits the engine; otherwise *out = nullptr and ISC_OK.
int line_build(const LayerIn *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes,
               LinePlan **out);
void line_free(LinePlan *p);

// Host only: 1 if the planner accepts the network (then *smem_bytes = shared memory per CTA), else 0 and *rule =
// the number of the rule that refused it.
int line_plan_probe(const LayerIn *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes, int *rule,
                    uint32_t *smem_bytes);

// Runs samples first..first+n-1 (ns.first_sample = first) and adds their votes to d_counts.
int line_run(LinePlan *p, const uint8_t *d_x, const NoiseStream &ns, int64_t n, int batch_hint,
             int32_t *d_counts, int8_t *d_logits, cudaStream_t st, int64_t *launches);

// Debug read-back: runs one group up to the phase producing model tensor `tensor` and returns that
// tensor of sample ns.first_sample as [C][H][W] int32 (host).
int line_debug_tensor(LinePlan *p, const uint8_t *d_x, const NoiseStream &ns, int tensor, int32_t *out_chw,
                      int32_t *d_counts_scratch, cudaStream_t st, int64_t *launches);

// After the stream has been synchronised: ISC_OK, or ISC_ERR_TIMEOUT if a bounded wait expired.
int line_check(LinePlan *p);

// Failure-path check without a failure: runs the engine's wait code (one thread) on a barrier and a counter that nothing
// completes, with `limit_ns` as the wait limit.  Returns what line_check returns afterwards (ISC_ERR_TIMEOUT when the
// path works) and out[] = {first wait's result, second wait's result, abort flag, nanoseconds spent}.
int line_wait_probe(LinePlan *p, long long limit_ns, int32_t out[4], cudaStream_t st);

// SM cycles, summed over CTAs and over every launch so far, spent in: [0] halo fills, [1] the noise phase (draw, add,
// saturate, store: Def. 3.3, Def. 3.4), [2] the convolutions, [3] pool / FC / argmax / vote.  Synchronises the device.
int line_phase_cycles(LinePlan *p, unsigned long long out[4]);

}  // namespace isc
