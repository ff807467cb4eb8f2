// Fill rate of the shared-memory tiles of the 8x8-region attention kernel: bulk tensor copies (TMA) against
// 16-byte cp.async copies, same bytes per tile, same CTAs per SM.  Own GPU memory only, no multicast.
#include <cstdio>
#include <cstdlib>
#include <cstdint>
#include <vector>
#include <cuda.h>
#include <cuda_runtime.h>

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %d\n", cudaGetErrorString(e_), __LINE__); exit(1); } } while (0)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}

constexpr int H = 56, W = 56, C = 64, S = 7, R = 49;
constexpr int OFF_Q = 0, OFF_K = 8192, OFF_V = 16384, OFF_HALO = 24576, OFF_BAR = 24576 + 18432, SMEM = OFF_BAR + 64 + 1024;

// MODE 0: seven boxes per tile (Q, K, V as two {32 ch, 8, 8} boxes each + the {64 ch, 12, 12} halo)
// MODE 1: four boxes per tile (Q, K, V as one {64 ch, 8, 8} box each + halo)
// MODE 2: halo box only; MODE 3: the six small boxes only
template <int MODE>
__global__ void __launch_bounds__(128, 4)
tma_kernel(const __grid_constant__ CUtensorMap mq32, const __grid_constant__ CUtensorMap mk32, const __grid_constant__ CUtensorMap mv32,
           const __grid_constant__ CUtensorMap mq64, const __grid_constant__ CUtensorMap mk64, const __grid_constant__ CUtensorMap mv64,
           const __grid_constant__ CUtensorMap mhalo, const int* __restrict__ route, int tiles, float* out) {
    extern __shared__ uint8_t raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bar = (uint64_t*)(smem + OFF_BAR);
    const uint32_t sb = smem_u32(smem);
    if (threadIdx.x == 0) { mbar_init(bar, 1); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
    __syncthreads();
    float acc = 0.f;
    uint32_t phase = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x) {
        const int b = t / R, i = t % R, y0 = (i / S) * 8, x0 = (i % S) * 8;
        if (threadIdx.x == 0) {
            const int ra = route[2 * t], rb = route[2 * t + 1];
            const int ya = (ra / S) * 8, xa = (ra % S) * 8, yb = (rb / S) * 8, xb = (rb % S) * 8;
            uint32_t bytes = 0;
            if (MODE == 0 || MODE == 3) bytes += 6 * 4096;
            if (MODE == 1) bytes += 3 * 8192;
            if (MODE != 3) bytes += 18432;
            mbar_expect_tx(bar, bytes);
            if (MODE == 0 || MODE == 3) {
                tma_load_4d(sb + OFF_Q, &mq32, bar, 0, x0, y0, b);
                tma_load_4d(sb + OFF_Q + 4096, &mq32, bar, 32, x0, y0, b);
                tma_load_4d(sb + OFF_K, &mk32, bar, 0, xa, ya, b);
                tma_load_4d(sb + OFF_K + 4096, &mk32, bar, 32, xb, yb, b);
                tma_load_4d(sb + OFF_V, &mv32, bar, 0, xa, ya, b);
                tma_load_4d(sb + OFF_V + 4096, &mv32, bar, 32, xb, yb, b);
            }
            if (MODE == 1) {
                tma_load_4d(sb + OFF_Q, &mq64, bar, 0, x0, y0, b);
                tma_load_4d(sb + OFF_K, &mk64, bar, 0, xa, ya, b);
                tma_load_4d(sb + OFF_V, &mv64, bar, 0, xa, ya, b);
            }
            if (MODE != 3) tma_load_4d(sb + OFF_HALO, &mhalo, bar, 0, x0 - 2, y0 - 2, b);
        }
        bool done = false;
        for (int it = 0; it < 4000000 && !done; ++it) done = mbar_try_wait(bar, phase);
        phase ^= 1;
        acc += *(float*)(smem + OFF_HALO + threadIdx.x * 128) + *(float*)(smem + threadIdx.x * 64);
        __syncthreads();
    }
    out[blockIdx.x * 128 + threadIdx.x] = acc;
}

__global__ void __launch_bounds__(128, 4)
cpasync_kernel(const uint8_t* __restrict__ Qb, const uint8_t* __restrict__ Kb, const uint8_t* __restrict__ Vb,
               const int* __restrict__ route, int tiles, float* out) {
    extern __shared__ uint8_t raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sb = smem_u32(smem);
    const int tid = threadIdx.x;
    const int c = tid & 7, tx = (tid >> 3) & 7, lrow = (tid >> 6) * 4, lhead = c >> 2;
    const uint32_t tile_off = lhead * 4096 + (lrow * 8 + tx) * 64 + (((c & 3) ^ ((tx >> 1) & 3)) << 4);
    const uint32_t v_off = (lrow * 8 + tx) * 128 + ((c ^ tx) << 4);
    const size_t row_bytes = (size_t)W * C * 2, img_bytes = (size_t)H * row_bytes;
    const size_t thr_off = (size_t)lrow * row_bytes + (size_t)tx * C * 2 + c * 16;
    const int hx = tid >> 3;
    float acc = 0.f;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x) {
        const int b = t / R, i = t % R, y0 = (i / S) * 8, x0 = (i % S) * 8;
        const int r = route[2 * t + lhead];
        const int yr = (r / S) * 8, xr = (r % S) * 8;
        const size_t qo = (size_t)b * img_bytes + (size_t)y0 * row_bytes + (size_t)x0 * C * 2 + thr_off;
        const size_t ko = (size_t)b * img_bytes + (size_t)yr * row_bytes + (size_t)xr * C * 2 + thr_off;
#pragma unroll
        for (int u = 0; u < 4; ++u) cp_async_16(sb + OFF_Q + tile_off + u * 512, Qb + qo + u * row_bytes, 16);
#pragma unroll
        for (int u = 0; u < 4; ++u) cp_async_16(sb + OFF_K + tile_off + u * 512, Kb + ko + u * row_bytes, 16);
#pragma unroll
        for (int u = 0; u < 4; ++u) cp_async_16(sb + OFF_V + v_off + u * 1024, Vb + ko + u * row_bytes, 16);
        if (hx < 12) {
            const bool col_in = (x0 + hx >= 2) && (x0 + hx - 2 < W);
            const uint8_t* src = Vb + (size_t)b * img_bytes + (size_t)x0 * C * 2 + c * 16 + (ptrdiff_t)(hx - 2) * C * 2;
#pragma unroll
            for (int hy = 0; hy < 12; ++hy) {
                const int y = y0 + hy - 2;
                const bool inb = col_in && y >= 0 && y < H;
                cp_async_16(sb + OFF_HALO + tid * 16 + hy * 1536, inb ? src + (ptrdiff_t)y * (ptrdiff_t)row_bytes : Vb, inb ? 16u : 0u);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        acc += *(float*)(smem + OFF_HALO + threadIdx.x * 128) + *(float*)(smem + threadIdx.x * 64);
        __syncthreads();
    }
    out[blockIdx.x * 128 + threadIdx.x] = acc;
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static CUtensorMap make_map(EncodeFn enc, void* base, int B, int bc, int bx, int by, CUtensorMapSwizzle sw) {
    CUtensorMap m;
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    cuuint32_t box[4] = {(cuuint32_t)bc, (cuuint32_t)bx, (cuuint32_t)by, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = enc(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { printf("encode failed %d\n", (int)r); exit(1); }
    return m;
}

int main() {
    const int B = 192;                       // 77 MB per tensor: Q, K, V together exceed the L2
    const size_t tensor_bytes = (size_t)B * H * W * C * 2;
    uint8_t *q, *k, *v; int* route; float* out;
    CK(cudaMalloc(&q, tensor_bytes)); CK(cudaMalloc(&k, tensor_bytes)); CK(cudaMalloc(&v, tensor_bytes));
    CK(cudaMemset(q, 1, tensor_bytes)); CK(cudaMemset(k, 2, tensor_bytes)); CK(cudaMemset(v, 3, tensor_bytes));
    const int tiles = B * R;
    std::vector<int> hr(2 * tiles);
    uint32_t s = 12345;
    for (auto& x : hr) { s = s * 1664525u + 1013904223u; x = (s >> 8) % R; }
    CK(cudaMalloc(&route, hr.size() * 4)); CK(cudaMemcpy(route, hr.data(), hr.size() * 4, cudaMemcpyHostToDevice));
    CK(cudaMalloc(&out, 148 * 4 * 128 * 4));
    EncodeFn enc = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&enc, cudaEnableDefault, &qres));
    if (!enc) { printf("no cuTensorMapEncodeTiled\n"); return 1; }
    CUtensorMap mq32 = make_map(enc, q, B, 32, 8, 8, CU_TENSOR_MAP_SWIZZLE_64B), mk32 = make_map(enc, k, B, 32, 8, 8, CU_TENSOR_MAP_SWIZZLE_64B),
                mv32 = make_map(enc, v, B, 32, 8, 8, CU_TENSOR_MAP_SWIZZLE_64B);
    CUtensorMap mq64 = make_map(enc, q, B, 64, 8, 8, CU_TENSOR_MAP_SWIZZLE_128B), mk64 = make_map(enc, k, B, 64, 8, 8, CU_TENSOR_MAP_SWIZZLE_128B),
                mv64 = make_map(enc, v, B, 64, 8, 8, CU_TENSOR_MAP_SWIZZLE_128B);
    CUtensorMap mh = make_map(enc, v, B, 64, 12, 12, CU_TENSOR_MAP_SWIZZLE_NONE);
    CK(cudaFuncSetAttribute(tma_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
    CK(cudaFuncSetAttribute(tma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
    CK(cudaFuncSetAttribute(tma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
    CK(cudaFuncSetAttribute(tma_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
    CK(cudaFuncSetAttribute(cpasync_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    const char* names[5] = {"TMA 6 x {32ch,8,8} + halo {64,12,12}", "TMA 3 x {64ch,8,8} + halo", "TMA halo only (18 KB boxes)",
                            "TMA 6 x {32ch,8,8} only (4 KB boxes)", "cp.async 16 B, same tiles"};
    const double bytes_per_tile[5] = {42.0 * 1024, 42.0 * 1024, 18.0 * 1024, 24.0 * 1024, 42.0 * 1024};
    for (int ctas = 1; ctas <= 4; ++ctas) {
        if (ctas == 3) continue;
        for (int m = 0; m < 5; ++m) {
            float best = 1e9f;
            for (int rep = 0; rep < 4; ++rep) {
                cudaEventRecord(e0);
                const int grid = 148 * ctas;
                if (m == 0) tma_kernel<0><<<grid, 128, SMEM>>>(mq32, mk32, mv32, mq64, mk64, mv64, mh, route, tiles, out);
                if (m == 1) tma_kernel<1><<<grid, 128, SMEM>>>(mq32, mk32, mv32, mq64, mk64, mv64, mh, route, tiles, out);
                if (m == 2) tma_kernel<2><<<grid, 128, SMEM>>>(mq32, mk32, mv32, mq64, mk64, mv64, mh, route, tiles, out);
                if (m == 3) tma_kernel<3><<<grid, 128, SMEM>>>(mq32, mk32, mv32, mq64, mk64, mv64, mh, route, tiles, out);
                if (m == 4) cpasync_kernel<<<grid, 128, SMEM>>>(q, k, v, route, tiles, out);
                cudaEventRecord(e1);
                CK(cudaEventSynchronize(e1));
                float ms; cudaEventElapsedTime(&ms, e0, e1);
                if (rep > 0 && ms < best) best = ms;
            }
            printf("%d CTA/SM  %-40s %8.1f us  %7.0f GB/s into shared memory  (%.2f us per tile per CTA)\n", ctas, names[m], best * 1e3,
                   tiles * bytes_per_tile[m] / (best * 1e-3) / 1e9, best * 1e3 / (tiles / (148.0 * ctas)));
        }
    }
    CK(cudaGetLastError());
    printf("done\n");
    return 0;
}
