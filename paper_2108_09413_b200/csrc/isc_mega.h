// Shared-memory-resident tensor-core engine for CIFAR-shaped residual networks.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "isc.h"
#include "isc_internal.h"

namespace isc {

struct MegaPlan;

struct MegaLayerIn {           // one validated layer with host arrays
    isc_layer d;
    const int8_t *w;
    const int32_t *bias;
    const int32_t *mult;
    const int8_t *shift;
};

// Builds the plan when the network fits the engine; otherwise *out = nullptr and ISC_OK.
int mega_build(const MegaLayerIn *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes,
               MegaPlan **out);
void mega_free(MegaPlan *p);

// Runs samples first..first+n-1 (ns.first_sample = first) and adds their votes to d_counts.
int mega_run(MegaPlan *p, const uint8_t *d_x, const NoiseStream &ns, int64_t n, int batch_hint,
             int32_t *d_counts, int8_t *d_logits, cudaStream_t st, int64_t *launches);

// Debug read-back: runs one group up to the phase producing model tensor `tensor` and returns that
// tensor of sample ns.first_sample as [C][H][W] int32 (host).  ISC_ERR_UNSUPPORTED if the tensor is
// not held by this engine.
int mega_debug_tensor(MegaPlan *p, const uint8_t *d_x, const NoiseStream &ns, int tensor, int32_t *out_chw,
                      int32_t *d_counts_scratch, cudaStream_t st, int64_t *launches);

// After the stream has been synchronised: ISC_OK, or ISC_ERR_TIMEOUT if a bounded wait expired.
int mega_check(MegaPlan *p);

}  // namespace isc
