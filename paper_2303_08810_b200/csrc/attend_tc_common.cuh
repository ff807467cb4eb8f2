// Shared by the two tcgen05 attention kernels for regions of 8 x 8 tokens (head dim 32, heads in pairs):
// shared-memory map, tile coordinates, small device helpers, and the argument block of the one-launch
// forward.
#pragma once

#include "bra_internal.h"
#include "sm100_ptx.cuh"

namespace bra {

using namespace ptx;

namespace tc {
constexpr int RS = 8;            // region side in tokens
constexpr int HALO = RS + 4;     // 12: region plus the 2-token LCE border
constexpr int THREADS = 128;
constexpr int KCAP = 64;         // largest topk
constexpr int TMEM_COLS = 128;   // S [0,128) fp32; then P [0,32) bf16 pairs + O [64,128)
constexpr int TM_O = 64;
constexpr int HALO_BYTES = HALO * HALO * 128;            // 18432
// shared memory map (bytes, from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                                 // [128 rows][64 B]  64B swizzle, K-major
constexpr int OFF_K = 8192;                              // [128 keys][64 B]  64B swizzle, K-major (buffer 0)
constexpr int OFF_V = 16384;                             // [64 keys][128 B]  128B swizzle, MN-major (buffer 0)
constexpr int OFF_ST = OFF_V;                            // [64 tokens][64 ch] fp32 staging: over V (buffer 0) + scratch
constexpr int OFF_POOL = 24576;                          // second half of the staging tile; scratch of the one-launch forward (pooling partial sums, K^r of a head)
constexpr int OFF_HALO = 32768;                          // [12][12][64 ch] bf16, linear
constexpr int OFF_BAR = OFF_HALO + HALO_BYTES;           // 51200: two mbarriers, tmem slot, job slots
constexpr int OFF_MISC = OFF_BAR + 64;                   // 1 KB: routing step, best key per (half, row)
constexpr int OFF_KV1 = 53248;                           // topk > 1 only: K buffer 1 (8 KB), V buffer 1 (8 KB)
constexpr int SMEM_K1 = OFF_MISC + 1024 + 1024;          // + slack for the manual 1024-byte alignment
constexpr int SMEM_KN = OFF_KV1 + 16384 + 1024;
static_assert(OFF_KV1 % 1024 == 0 && OFF_KV1 >= OFF_MISC + 1024, "buffer 1 placement");
constexpr uint32_t POLL_LIMIT = 4000000u;
constexpr uint32_t FLAG_POLLS = 1u << 20;                // polls of a grid-wide barrier, x ~0.2-0.5 us each: a fraction of a second
}  // namespace tc

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint4 ldg_nc_u4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ int32_t ld_acquire_gpu(const int32_t* p) {
    int32_t v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(int32_t* p, int32_t v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// order-preserving bits of an fp32 score (-0 and +0 tie), as in the stand-alone routing kernels
__device__ __forceinline__ uint32_t score_bits(float s) {
    s += 0.0f;
    const uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct TileCoord { int b, i, hp, y0, x0, c0; };
// Walks tiles T, T + stride, ... (T = (b * R + i) * pairs + hp) with adds and carries only.
struct TileWalker {
    int pairs, R;
    int d_hp, d_i, d_b;                // stride split into (hp, i, b) digits
    int hp, i, b;
    __device__ __forceinline__ void init(int T, int stride, const Dims& dm) {
        pairs = dm.heads >> 1; R = dm.R;
        hp = T % pairs; i = (T / pairs) % R; b = T / (pairs * R);
        d_hp = stride % pairs; d_i = (stride / pairs) % R; d_b = stride / (pairs * R);
    }
    __device__ __forceinline__ void next() {
        hp += d_hp;
        int carry = hp >= pairs;
        hp -= carry ? pairs : 0;
        i += d_i + carry;
        carry = i >= R;
        i -= carry ? R : 0;
        b += d_b + carry;
    }
};

// the topk = 1 kernel (attend_tc_k1.cu); launch_attend_tc() forwards to it
cudaError_t launch_attend_tc_k1(const Dims& d, const void* Q, const void* K, const void* V,
                                const int32_t* index, const float* lce_w, const float* lce_b,
                                void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel);

inline int tc_sm_count() {
    int dev = 0, n = 1;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 1;
    return n;
}

}  // namespace bra
