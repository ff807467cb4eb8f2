// bra_route_static: region-to-region routing for callers that cannot supply
// scratch memory.  The region means that bra_route keeps in the caller's
// workspace live here in an array that is part of the library image, so the
// call neither needs nor performs any allocation.
#include "bra_internal.h"

#include <mutex>

namespace bra {

// Q^r in the first half, K^r in the second.  Present on every device that
// loads the library, for the life of the process.
static __device__ __align__(256) float g_route_means[2 * BRA_ROUTE_STATIC_MAX_MEAN_FLOATS];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_lock;
float* g_means_addr[kMaxDevices] = {};   // device address of g_route_means, per device ordinal

// In host code `g_route_means` names a host-side shadow of the symbol, not
// device memory: the kernels must be given the address the runtime reports
// for the device that is current.  Looked up once per device.
bra_status means_address(float** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BRA_ERR_CUDA;
    std::lock_guard<std::mutex> guard(g_lock);
    if (!g_means_addr[dev]) {
        float* addr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), g_route_means) != cudaSuccess || !addr)
            return BRA_ERR_CUDA;
        g_means_addr[dev] = addr;
    }
    *out = g_means_addr[dev];
    return BRA_OK;
}
}  // namespace
}  // namespace bra

using namespace bra;

extern "C" bra_status bra_route_static(const bra_problem* p, const void* Q, const void* K,
                                       int32_t* index, void* stream) {
    reset_launch_count();
    Dims d;
    bra_status s = check_problem(p, &d);
    if (s != BRA_OK) return s;
    if (!Q || !K || !index) return BRA_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) |
         reinterpret_cast<uintptr_t>(index)) & 15) return BRA_ERR_ALIGN;
    const size_t mean_floats = (size_t)d.B * d.R * d.C;
    if (mean_floats > (size_t)BRA_ROUTE_STATIC_MAX_MEAN_FLOATS) return BRA_ERR_STATIC_LIMIT;
    if (!route_supported(d)) return BRA_ERR_UNSUPPORTED;
    if (d.H != d.H0 || d.W != d.W0) return BRA_ERR_UNSUPPORTED;      // a padded copy of Q and K would need scratch
    float* means = nullptr;
    if ((s = means_address(&means)) != BRA_OK) return s;
    float* q_mean = means;
    float* k_mean = means + BRA_ROUTE_STATIC_MAX_MEAN_FLOATS;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // pooling writes every element of both mean tensors that routing reads: no clearing needed
    if (launch_pool(d, p->dtype, Q, K, q_mean, k_mean, st) != cudaSuccess) return BRA_ERR_CUDA;
    if (launch_route(d, q_mean, k_mean, index, st) != cudaSuccess) return BRA_ERR_CUDA;
    return BRA_OK;
}
