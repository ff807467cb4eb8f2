// Internal declarations shared by the translation units of the BRA library.
// Nothing here is part of the C boundary (include/bra.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>

#include <mutex>

#include "../../include/bra.h"

namespace bra {

// Problem with every derived quantity the kernels need, passed by value.
struct Dims {
    int B, H, W, C, heads, S, topk;
    int d;        // C / heads
    int R;        // S * S regions
    int hs, ws;   // region height / width in tokens
    int n_r;      // hs * ws tokens per region
    int N;        // H * W tokens per image
    int heads_i;  // heads of the routing index: heads, or 1 with shared routing
    int lce;      // 1: add LCE
    float scale;  // softmax scale (Eq. 1)
    // When S does not divide the caller's map, H and W above are the padded sizes (next multiples of S: the
    // kernels only ever see a divisible map) and these are the caller's; equal to H, W otherwise.
    int H0, W0;
    int esize;    // bytes per element of Q, K, V, O
};

// Scratch layout (byte offsets from ws, all multiples of 256).
struct WsLayout {
    size_t status;      // int32[64]: [0] first device error, [1] detail
    size_t q_mean;      // fp32 [B,R,C]
    size_t k_mean;      // fp32 [B,R,C]
    size_t index;       // int32 [B,heads_i,R,topk] (bra_forward with index == NULL)
    size_t delta;       // fp32 [B,heads,N]  rowsum(P o dP) of the backward pass
    size_t inv_off;     // int32 [B,heads_i,R+1] CSR offsets of the inverse routing index
    size_t inv_list;    // int32 [B,heads_i,R*topk] query regions routed to each key region
    size_t dw_part;     // fp32 [dw_blocks, C*26] partial LCE weight / bias gradients
    size_t pad;         // padded maps only: seven [B,H,W,C] tensors of the padded size (Q, K, V, O / dO, dQ, dK, dV)
    size_t pad_lse;     // padded maps only: fp32 [B,heads,H*W] of the padded size
    size_t pad_tensor;  // bytes of one padded tensor
    size_t total;
    int dw_blocks;
};

WsLayout ws_layout(const Dims& d);

// Host-side bookkeeping of kernel launches for bra_last_launch_count().
void count_launch(int n = 1);
void reset_launch_count();

// Validate a problem statement and fill the derived dimensions.
bra_status check_problem(const bra_problem* p, Dims* out);

// ---- kernel launchers (each returns the cudaError of its launches) ----------
// Copies between the caller's [B,H0,W0,C] map and the zero-padded [B,H,W,C] map the kernels work on
// (to_padded: fill; else crop).  elem_bytes: bytes of one token (C * element size; a multiple of 4).
cudaError_t launch_pad_copy(const void* src, void* dst, long long images, int H0, int W0, int H, int W,
                            int token_bytes, bool to_padded, cudaStream_t st);
cudaError_t launch_pool(const Dims& d, int dtype, const void* Q, const void* K,
                        float* q_mean, float* k_mean, cudaStream_t st);
cudaError_t launch_route(const Dims& d, const float* q_mean, const float* k_mean,
                         int32_t* index, cudaStream_t st);
// true if this build has a routing kernel for the problem
bool route_supported(const Dims& d);

bool attend_simt_supported(const Dims& d);
cudaError_t launch_attend_simt(const Dims& d, int dtype, const void* Q, const void* K, const void* V,
                               const int32_t* index, const float* lce_w, const float* lce_b,
                               void* O, float* lse, int32_t* status, cudaStream_t st);

bool attend_mma_supported(const Dims& d, int dtype);
cudaError_t launch_attend_mma(const Dims& d, const void* Q, const void* K, const void* V,
                              const int32_t* index, const float* lce_w, const float* lce_b,
                              void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel);

// after_own_kernel (here and below): the kernel before this one in the stream is the library's own
// routing kernel, so the launch may overlap its tail (programmatic dependent launch)
bool attend_tc_supported(const Dims& d, int dtype);
cudaError_t launch_attend_tc(const Dims& d, const void* Q, const void* K, const void* V,
                             const int32_t* index, const float* lce_w, const float* lce_b,
                             void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel);

// Algorithm 1 in one launch (pooling, routing and attention of 8 x 8-token regions, topk = 1)
bool forward_tc_supported(const Dims& d, int dtype);
cudaError_t launch_forward_tc(const Dims& d, const void* Q, const void* K, const void* V,
                              const float* lce_w, const float* lce_b, void* O, int32_t* index, float* lse,
                              float* q_mean, float* k_mean, int32_t* ctrl, int inject, cudaStream_t st);

bool attend_img_supported(const Dims& d, int dtype);
cudaError_t launch_attend_img(const Dims& d, const void* Q, const void* K, const void* V,
                              const int32_t* index, const float* lce_w, const float* lce_b,
                              void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel);
bool attend_tc_wide_supported(const Dims& d, int dtype);
cudaError_t launch_attend_tc_wide(const Dims& d, const void* Q, const void* K, const void* V,
                                  const int32_t* index, const float* lce_w, const float* lce_b,
                                  void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel);

bool backward_mma_supported(const Dims& d, int dtype);
cudaError_t launch_backward_mma(const Dims& d, const void* Q, const void* K, const void* V,
                                const int32_t* index, const int32_t* inv_off, const int32_t* inv_list,
                                const float* lce_w, const float* lse, const void* dO,
                                void* dQ, void* dK, void* dV, float* delta, int32_t* status, cudaStream_t st);

bool backward_img_supported(const Dims& d, int dtype);
cudaError_t launch_backward_img(const Dims& d, const void* Q, const void* K, const void* V,
                                const int32_t* index, const int32_t* inv_off, const int32_t* inv_list,
                                const float* lce_w, const float* lse, const void* dO,
                                void* dQ, void* dK, void* dV, float* delta, int32_t* status, cudaStream_t st);

// A process may drive several GPUs, and kernel attributes are per device: the largest value already
// set for a kernel on the CURRENT device (dynamic shared-memory size, or 1 for "set-up done").  The
// set-up runs under a lock and is recorded only once it has succeeded, so concurrent host threads
// never launch before the attribute exists and a failed set-up is tried again.
struct PerDeviceMax {
    std::mutex lock;
    int v[64] = {};
    template <typename F>
    cudaError_t ensure(int want, F&& set) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return set();
        std::lock_guard<std::mutex> guard(lock);
        if (want <= v[dev]) return cudaSuccess;
        const cudaError_t e = set();
        if (e == cudaSuccess) v[dev] = want;
        return e;
    }
};
struct PerDeviceOnce {
    PerDeviceMax m;
    template <typename F>
    cudaError_t run(F&& set) { return m.ensure(1, set); }
};

// A helper stream per device and host thread, forked from and joined back into the caller's stream with
// events (created on first use; nullptr if that fails or BRA_NO_SIDE_STREAM is set: then the work stays in
// order on the caller's stream).
struct SideStream { cudaStream_t s; cudaEvent_t fork, join; };
SideStream* side_stream();

bool backward_supported(const Dims& d);
// impl: the bra_impl the caller asked for
cudaError_t launch_backward(const Dims& d, int dtype, int impl, const void* Q, const void* K, const void* V,
                            const int32_t* index, const float* lce_w, const float* lse,
                            const void* dO, void* dQ, void* dK, void* dV,
                            float* d_lce_w, float* d_lce_b,
                            char* ws, const WsLayout& L, cudaStream_t st);

// ---- device helpers -----------------------------------------------------------
#ifdef __CUDACC__
// Programmatic dependent launch: a kernel launched with launch_kernel(..., after_own_kernel = true)
// may start while the kernel before it in the stream is still running; pdl_wait() returns once
// that kernel has completed and its writes are visible (a no-op for an ordinary launch).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 bool after_own_kernel, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    static const bool pdl_off = getenv("BRA_NO_PDL") != nullptr;   // debugging aid: plain stream order
    cfg.numAttrs = (after_own_kernel && !pdl_off) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ void record_error(int32_t* status, int code, int detail) {
    if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

// Load `n` consecutive elements (n multiple of 8 for bf16 / 4 for fp32, 16-byte aligned) as fp32.
template <int n>
__device__ __forceinline__ void load_row(const float* __restrict__ p, float* out) {
#pragma unroll
    for (int i = 0; i < n; i += 4) {
        float4 v = __ldg(reinterpret_cast<const float4*>(p + i));
        out[i] = v.x; out[i + 1] = v.y; out[i + 2] = v.z; out[i + 3] = v.w;
    }
}
template <int n>
__device__ __forceinline__ void load_row(const __nv_bfloat16* __restrict__ p, float* out) {
#pragma unroll
    for (int i = 0; i < n; i += 8) {
        uint4 v = __ldg(reinterpret_cast<const uint4*>(p + i));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            out[i + 2 * j] = __uint_as_float(w[j] << 16);
            out[i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
    }
}
template <int n>
__device__ __forceinline__ void store_row(float* p, const float* v) {
#pragma unroll
    for (int i = 0; i < n; i += 4)
        *reinterpret_cast<float4*>(p + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
}
template <int n>
__device__ __forceinline__ void store_row(__nv_bfloat16* p, const float* v) {
#pragma unroll
    for (int i = 0; i < n; i += 8) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            __nv_bfloat162 h = __floats2bfloat162_rn(v[i + 2 * j], v[i + 2 * j + 1]);
            w[j] = *reinterpret_cast<uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p + i) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}
#endif  // __CUDACC__

}  // namespace bra
