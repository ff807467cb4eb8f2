// Cost per tcgen05.mma instruction (M = 128, K = 16, bf16) for the operand forms the attention kernels use:
// one thread issues `reps` MMAs into the same accumulator, commits, waits (bounded); clock64() around it.
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include "../sm100_ptx.cuh"
using namespace bra::ptx;

// MODE 0: A, B from shared memory (K-major, 64-byte swizzle), N columns.  MODE 1: A from tensor memory, B = [keys][64 B] MN-major, N = 32.
template <int MODE, int N>
__global__ void __launch_bounds__(128, 1) k(long long* cyc, int reps, int* err) {
    extern __shared__ uint8_t raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + 40960);
    uint32_t* slot = reinterpret_cast<uint32_t*>(bar + 1);
    for (int i = threadIdx.x; i < 40960 / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0x3c003c00u;   // small bf16 values
    if (threadIdx.x == 0) { mbar_init(bar, 1); fence_mbar_init(); }
    if (threadIdx.x < 32) tmem_alloc(slot, 512);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *slot;
    const uint32_t base = smem_u32(smem);
    bool ok = true;
    if (threadIdx.x == 0) {
        constexpr uint32_t IS = umma_idesc_bf16(128, N, false, false);
        constexpr uint32_t IO = umma_idesc_bf16(128, 32, false, true);
        long long t0 = clock64();
        for (int r = 0; r < reps; ++r) {
            if (MODE == 0) umma_ss(tmem, umma_smem_desc(base + (r & 1) * 32, 16, 512, 4), umma_smem_desc(base + 8192 + (r & 1) * 32, 16, 512, 4), IS, r);
            else umma_ts(tmem + 256, tmem + (r & 7) * 8, umma_smem_desc(base + 8192, 16, 512, 4) + (uint64_t)((r & 7) * 64), IO, r);
        }
        umma_commit(bar);
        long long t1 = clock64();
        ok = mbar_wait(bar, 0, 4000000u);
        long long t2 = clock64();
        cyc[blockIdx.x * 2] = t1 - t0;
        cyc[blockIdx.x * 2 + 1] = t2 - t0;
        if (!ok) *err = 1;
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) { tc_fence_after_sync(); tmem_dealloc(tmem, 512); }
}

template <int MODE, int N>
void run(const char* name, long long* cyc, int* err, int sms) {
    cudaFuncSetAttribute(k<MODE, N>, cudaFuncAttributeMaxDynamicSharedMemorySize, 43008);
    for (int reps : {8, 64, 256}) {
        k<MODE, N><<<sms, 128, 43008>>>(cyc, reps, err);
        k<MODE, N><<<sms, 128, 43008>>>(cyc, reps, err);
        cudaDeviceSynchronize();
        long long h[2];
        cudaMemcpy(h, cyc, sizeof(h), cudaMemcpyDeviceToHost);
        printf("%-34s reps %3d: issue %6lld cycles, done after %6lld cycles  (%.1f per MMA)\n", name, reps, h[0], h[1], (double)h[1] / reps);
    }
}

int main() {
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    long long* cyc; int* err;
    cudaMalloc(&cyc, sizeof(long long) * 2 * sms);
    cudaMalloc(&err, sizeof(int));
    cudaMemset(err, 0, sizeof(int));
    run<0, 32>("A,B smem  N=32", cyc, err, sms);
    run<0, 64>("A,B smem  N=64", cyc, err, sms);
    run<0, 128>("A,B smem  N=128", cyc, err, sms);
    run<0, 256>("A,B smem  N=256", cyc, err, sms);
    run<1, 32>("A tmem, B smem MN-major  N=32", cyc, err, sms);
    int h = 0;
    cudaMemcpy(&h, err, sizeof(int), cudaMemcpyDeviceToHost);
    cudaError_t e = cudaDeviceSynchronize();
    printf("status %s, timeouts %d\n", cudaGetErrorString(e), h);
    return e != cudaSuccess || h;
}
