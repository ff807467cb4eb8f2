// placeholder until the TMA + tcgen05 kernel lands
#include "bra_internal.h"
namespace bra {
bool attend_tc_supported(const Dims&, int) { return false; }
cudaError_t launch_attend_tc(const Dims&, const void*, const void*, const void*, const int32_t*,
                             const float*, const float*, void*, float*, int32_t*, cudaStream_t) {
    return cudaErrorNotSupported;
}
}
