// placeholder until the warp-level tensor-core kernel lands
#include "bra_internal.h"
namespace bra {
bool attend_mma_supported(const Dims&, int) { return false; }
cudaError_t launch_attend_mma(const Dims&, const void*, const void*, const void*, const int32_t*,
                              const float*, const float*, void*, float*, int32_t*, cudaStream_t) {
    return cudaErrorNotSupported;
}
}
