// Throughput of single instructions per SM and clock: one CTA of 512 threads per SM, eight independent
// dependency chains per thread, clock64() around the loop.  The instructions are the ones the softmax and
// the LCE of the attention kernels are made of.
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_bf16.h>

template <int OP>
__global__ void __launch_bounds__(512, 1) k(float* out, long long* cyc, int iters, float seed) {
    float a[8];
    uint32_t u[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { a[i] = seed + threadIdx.x * 1e-3f + i * 0.125f; u[i] = threadIdx.x + i; }
    __syncthreads();
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (OP == 0) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(a[i]));
            if (OP == 1) asm volatile("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(u[i]) : "f"(a[i]), "f"(a[(i + 1) & 7]));
            if (OP == 2) asm volatile("fma.rn.f32 %0, %0, %1, %1;" : "+f"(a[i]) : "f"(seed));
            if (OP == 3) { asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(a[i])); asm volatile("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(u[i]) : "f"(a[i]), "f"(a[(i + 1) & 7])); }
            if (OP == 4) asm volatile("{.reg .b64 t, s; mov.b64 t, {%0, %1}; mov.b64 s, {%2, %2}; fma.rn.f32x2 t, t, s, s; mov.b64 {%0, %1}, t;}" : "+f"(a[i]), "+f"(a[(i + 4) & 7]) : "f"(seed));
            if (OP == 5) asm volatile("max.f32 %0, %0, %1, %2;" : "+f"(a[i]) : "f"(a[(i + 1) & 7]), "f"(seed));
            if (OP == 6) asm volatile("lg2.approx.ftz.f32 %0, %0;" : "+f"(a[i]));
            if (OP == 7) { asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(a[i])); asm volatile("fma.rn.f32 %0, %0, %1, %1;" : "+f"(a[(i + 3) & 7]) : "f"(seed)); }
            if (OP == 8) asm volatile("shl.b32 %0, %0, 16;" : "+r"(u[i]));
            if (OP == 9) asm volatile("and.b32 %0, %0, 0xffff0000;" : "+r"(u[i]));
            if (OP == 10) asm volatile("prmt.b32 %0, %0, 0, 0x1044;" : "+r"(u[i]));
            if (OP == 11) asm volatile("add.rn.f32x2 %0, %0, %1;" : "+l"(*reinterpret_cast<unsigned long long*>(&a[2 * (i & 3)])) : "l"(*reinterpret_cast<unsigned long long*>(&a[2 * ((i + 1) & 3)])));
        }
    }
    long long t1 = clock64();
    float s = 0.f;
    uint32_t x = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { s += a[i]; x ^= u[i]; }
    out[blockIdx.x * blockDim.x + threadIdx.x] = s + __uint_as_float(x & 0xff);
    if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}

template <int OP>
void run(const char* name, int per_iter_ops, float* out, long long* cyc, int sms) {
    const int iters = 4096;
    k<OP><<<sms, 512>>>(out, cyc, iters, 0.5f);
    k<OP><<<sms, 512>>>(out, cyc, iters, 0.5f);
    cudaDeviceSynchronize();
    long long h[256];
    cudaMemcpy(h, cyc, sizeof(long long) * sms, cudaMemcpyDeviceToHost);
    long long mx = 0;
    for (int i = 0; i < sms; ++i) mx = h[i] > mx ? h[i] : mx;
    double thread_ops = (double)iters * 8 * per_iter_ops * 512;
    printf("%-28s %8.2f thread-ops / clk / SM   (%lld cycles)\n", name, thread_ops / (double)mx, mx);
}

int main() {
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    float* out; long long* cyc;
    cudaMalloc(&out, sizeof(float) * 512 * sms);
    cudaMalloc(&cyc, sizeof(long long) * sms);
    run<0>("ex2.approx.ftz.f32", 1, out, cyc, sms);
    run<6>("lg2.approx.ftz.f32", 1, out, cyc, sms);
    run<3>("ex2 + cvt.bf16x2 (pairs)", 2, out, cyc, sms);
    run<2>("fma.rn.f32", 1, out, cyc, sms);
    run<4>("fma.rn.f32x2 (instr)", 1, out, cyc, sms);
    run<7>("ex2 + fma (pairs)", 2, out, cyc, sms);
    run<5>("max.f32 3-input", 1, out, cyc, sms);
    run<10>("prmt.b32", 1, out, cyc, sms);
    run<11>("add.rn.f32x2 (instr)", 1, out, cyc, sms);
    cudaError_t e = cudaDeviceSynchronize();
    printf("status %s\n", cudaGetErrorString(e));
    return e != cudaSuccess;
}
