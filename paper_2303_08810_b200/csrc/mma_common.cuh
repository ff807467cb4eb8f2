// Shared by the warp-level tensor-core kernels (forward and backward): geometry of a
// (image, region, head) group, fast division, ldmatrix / mma.sync wrappers.
#pragma once

#include "bra_internal.h"
#include "sm100_ptx.cuh"

namespace bra {

namespace wm {
constexpr int KB = 64;          // keys per block
constexpr int MAXW = 8;         // warps per CTA at most (128 query rows)
constexpr int KCAP = 256;       // largest topk
}  // namespace wm

struct MmaGeom {
    int nw;            // warps per CTA
    int chunks;        // token chunks per region
    int nblocks;       // key blocks per group = ceil(topk * n_r / 64)
    int stages;        // K/V buffers (1 or 2)
    int halo_w;        // ws + 4
    int halo_rows;     // rows of the halo tile (largest chunk) incl. the 4 border rows
    uint32_t mul_nr, mul_ws, mul_s;   // ceil(2^32 / d) for d = n_r, ws, S
    int off_q, off_kv, off_flag, off_idx, off_halo, smem_bytes;
    int planes;        // 32-channel planes of a head (head dim / 32); every tile below exists once per plane
};

__device__ __forceinline__ uint32_t fdiv(uint32_t n, uint32_t d, uint32_t mul) {
    return d == 1 ? n : __umulhi(n, mul);
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t* r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t* r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (fp32) += A (bf16, 16x16) * B (bf16, 16x8)
__device__ __forceinline__ void mma_bf16(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// D (fp32) = A * B (no accumulator to clear beforehand)
__device__ __forceinline__ void mma_bf16_zero(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%10, %10, %10, %10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}


// ------------------------------------------------------------------ host side
inline uint32_t recip32(int d) { return d <= 1 ? 0u : (uint32_t)(((1ull << 32) + (uint64_t)d - 1) / (uint64_t)d); }

inline MmaGeom mma_geom(const Dims& d, int planes = 1) {
    MmaGeom g;
    g.planes = planes;
    const int rb = (d.n_r + 15) / 16;
    g.nw = rb < wm::MAXW ? rb : wm::MAXW;
    g.chunks = (d.n_r + g.nw * 16 - 1) / (g.nw * 16);
    g.nblocks = (d.topk * d.n_r + wm::KB - 1) / wm::KB;
    g.stages = g.nblocks > 1 ? 2 : 1;
    g.halo_w = d.ws + 4;
    const int chunk_rows = (g.nw * 16 + d.ws - 1) / d.ws + 1;         // rows a chunk of tokens can touch
    g.halo_rows = (chunk_rows < d.hs ? chunk_rows : d.hs) + 4;
    g.mul_nr = recip32(d.n_r); g.mul_ws = recip32(d.ws); g.mul_s = recip32(d.S);
    int off = 0;
    g.off_q = off;    off += planes * g.nw * 16 * 64;
    g.off_kv = off;   off += planes * g.stages * 8192;                // also the fp32 staging tile: nw * 2 KB per plane
    g.off_flag = off; off += g.stages * wm::KB;
    g.off_idx = off;  off += ((d.topk * 4 + 15) / 16) * 16;
    g.off_halo = off; off += d.lce ? planes * g.halo_rows * g.halo_w * 64 : 0;
    g.smem_bytes = off;
    return g;
}


}  // namespace bra
