#include "isc_mega.h"

namespace isc {

struct MegaPlan { int unused; };

int mega_build(const MegaLayerIn *, int, int, int, int, int, MegaPlan **out)
{
    *out = nullptr;
    return ISC_OK;
}
void mega_free(MegaPlan *p) { delete p; }
int mega_run(MegaPlan *, const uint8_t *, const NoiseStream &, int64_t, int, int32_t *, int8_t *, cudaStream_t,
             int64_t *)
{
    return ISC_ERR_UNSUPPORTED;
}
int mega_check(MegaPlan *) { return ISC_OK; }

}  // namespace isc
