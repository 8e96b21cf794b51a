// tcgen05 / TMA (sm_100a) prefill path.
#include "gta_sm100.cuh"

namespace gta {

bool sm100_prefill_supported(const Dims&, int) { return false; }

gta_status_t launch_sm100_prefill(const Dims&, const void*, const void*, const void*, const void*, const void*,
                                  const void*, void*, void*, int32_t*, cudaStream_t, int, int*) {
    return GTA_ERR_UNSUPPORTED;
}

}  // namespace gta
