// Shared by the kernels that keep a whole (image, head) slice resident in shared memory
// (forward and backward): the slice layout, its loader, and the 5 x 5 depthwise correlation
// (LCE, or its adjoint with the flipped filter) read from a resident slice.
//
// Slice layout: token t of the image at byte t * 64 (the head's 32 bf16 channels), its four
// 16-byte chunks xor-swizzled with (t >> 1) & 3 so that ldmatrix over gathered token rows and
// the per-channel-pair reads of the correlation are both free of bank conflicts.
#pragma once

#include "mma_common.cuh"

namespace bra {

namespace img {
constexpr int KB = 64;            // keys (or columns) per block
constexpr int MAX_ENTRIES = 8192; // routing entries of one (image, head): R * topk
}  // namespace img

// cp.async the head's 64-byte slice of all N tokens of an image (src: the image's first token,
// already offset to the head's channels) to shared memory at dst.
__device__ __forceinline__ void img_load_slice(uint32_t dst, const uint8_t* src, int N, size_t tok_bytes,
                                               int tid, int nthreads) {
    for (int c = tid; c < N * 4; c += nthreads) {
        const int tok = c >> 2, q = c & 3;
        ptx::cp_async_16(dst + tok * 64 + ((q ^ ((tok >> 1) & 3)) << 4), src + (size_t)tok * tok_bytes + q * 16, 16);
    }
}

// [tap][channel pair] float2 table of the head's 5 x 5 weights in shared memory; flip: the adjoint's filter
__device__ __forceinline__ void img_load_weights(uint8_t* dst, const float* w_head, bool flip, int tid, int nthreads) {
    for (int idx = tid; idx < 25 * 16; idx += nthreads) {
        const int q = idx >> 4, cp = idx & 15;
        const int tap = flip ? 24 - q : q;
        *reinterpret_cast<float2*>(dst + idx * 8) =
            make_float2(__ldg(w_head + (2 * cp) * 25 + tap), __ldg(w_head + (2 * cp + 1) * 25 + tap));
    }
}

__device__ __forceinline__ uint32_t ldg_u32(const uint8_t* p) {
    return __ldg(reinterpret_cast<const uint32_t*>(p));
}


// 5 x 5 depthwise correlation (LCE) of the resident V slice for a block of BR rows x WS columns of
// tokens whose top-left token is (y, x) of the map, for one channel pair: sums added into acc.
// WS and x are even, so the tokens of a window row pair up on one swizzle phase: one address per
// pair of loads.  BORDER: the 2-token frame of the block may leave the map (zeros there).
template <int WS, int BR, bool BORDER>
__device__ __forceinline__ void lce_block(uint32_t vbase, int y, int x, int H, int W, int cq, uint32_t vcol,
                                          uint32_t wlane, float2 (*acc)[WS]) {
    constexpr int WW = WS + 4;
#pragma unroll
    for (int yy = 0; yy < BR + 4; ++yy) {
        const int iy = y + yy - 2;
        const bool row_ok = !BORDER || (unsigned)iy < (unsigned)H;
        const int rt = iy * W + x - 2;                       // token id of the window row's first column
        float2 v[WW];
#pragma unroll
        for (int j = 0; j < WW / 2; ++j) {
            const int tok = rt + 2 * j;                      // even: tok and tok + 1 share (tok >> 1) & 3
            const uint32_t a = vbase + tok * 64 + ((cq ^ ((tok >> 1) & 3)) << 4) + vcol;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int ix = x + 2 * j + e - 2;
                uint32_t w = 0u;
                if (row_ok && (!BORDER || (unsigned)ix < (unsigned)W)) w = ptx::lds_u32(a + e * 64);
                v[2 * j + e] = make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
            }
        }
        // window row yy meets tap rows ti = yy - r of the block's rows r: their weights come from the table
        // (wlane: this lane's channel pair) when they are needed, not held in registers throughout
#pragma unroll
        for (int ti = 0; ti < 5; ++ti) {
            const int r = yy - ti;
            if (r < 0 || r >= BR) continue;
            float2 w[5];
#pragma unroll
            for (int tj = 0; tj < 5; ++tj) w[tj] = ptx::lds_f32x2(wlane + (ti * 5 + tj) * 128);
#pragma unroll
            for (int tj = 0; tj < 5; ++tj)
#pragma unroll
                for (int c = 0; c < WS; ++c) acc[r][c] = __ffma2_rn(w[tj], v[c + tj], acc[r][c]);
        }
    }
}

// One lane's share of a unit whose 16 (or 4) tokens form full region rows: BR rows x WS columns from
// row r0 of the tile; adds the parked O^att and stores bf16.
// ONE_PATH: only the bounds-checked code (smaller; for kernels that are short of instruction cache).
template <int WS, int BR, bool ONE_PATH>
__device__ __forceinline__ void lce_store_block(uint32_t vbase, const float* stage_o, uint32_t* outb, int r0,
                                                int y0, int x0, const Dims& dm, int cp, bool lce,
                                                uint32_t wlane, float2 bias2) {
    float2 acc[BR][WS];
#pragma unroll
    for (int r = 0; r < BR; ++r)
#pragma unroll
        for (int c = 0; c < WS; ++c) acc[r][c] = bias2;
    const int y = y0 + r0, x = x0;
    if (lce) {
        const bool inside = y >= 2 && y + BR + 1 < dm.H && x >= 2 && x + WS + 1 < dm.W;
        if (!ONE_PATH && inside) lce_block<WS, BR, false>(vbase, y, x, dm.H, dm.W, cp >> 2, (cp & 3) * 4, wlane, acc);
        else        lce_block<WS, BR, true>(vbase, y, x, dm.H, dm.W, cp >> 2, (cp & 3) * 4, wlane, acc);
    }
#pragma unroll
    for (int r = 0; r < BR; ++r)
#pragma unroll
        for (int c = 0; c < WS; ++c) {
            const float2 att = *reinterpret_cast<const float2*>(stage_o + ((r0 + r) * WS + c) * 32 + 2 * cp);
            const float2 r2 = __fadd2_rn(att, acc[r][c]);
            outb[((size_t)(y + r) * dm.W + x + c) * (dm.C / 2)] = pack2_bf16(r2.x, r2.y);
        }
}


// One warp: out[token] = stage[token] + correlation of the resident slice at vbase with the weight
// table at wtab (shared-memory address; 0: no correlation), for the `rows` tokens from t0 of the
// region whose first token is (y0, x0); bf16 store of the head's 32 channels.  lane = (channel
// pair, half): whole region rows per half-warp for 4 x 4 and 2 x 2 regions, else runs along x.
// SHAPE: 44 = every region is 4 x 4 tokens, 22 = 2 x 2, 0 = anything (decided at launch: each
// instantiation carries one code path, which keeps the kernels inside the instruction cache).
template <int SHAPE, bool ONE_PATH = false>
__device__ __forceinline__ void img_lce_store(uint32_t vbase, uint32_t wtab, const float* stage_o, uint32_t* outb,
                                              int t0, int rows, int y0, int x0, const Dims& dm, uint32_t mul_ws,
                                              int lane, float2 bias2) {
    const int cp = lane & 15;
    const bool lce = wtab != 0u;
    if (SHAPE == 44) { lce_store_block<4, 2, ONE_PATH>(vbase, stage_o, outb, 2 * (lane >> 4), y0, x0, dm, cp, lce, wtab + cp * 8, bias2); return; }
    if (SHAPE == 22) { lce_store_block<2, 1, ONE_PATH>(vbase, stage_o, outb, lane >> 4, y0, x0, dm, cp, lce, wtab + cp * 8, bias2); return; }
    float2 wv[25];
    if (lce) {
#pragma unroll
        for (int q = 0; q < 25; ++q) wv[q] = ptx::lds_f32x2(wtab + (q * 16 + cp) * 8);
    }
    const uint32_t vcol = (cp & 3) * 4;
    const int cq = cp >> 2;
    const int run = (dm.ws & 1) ? 1 : 2;
    const int nruns = rows / run;                             // tiles start at multiples of 16, n_r is a multiple of run
    for (int u2 = lane >> 4; u2 < nruns; u2 += 2) {
        const int t = t0 + u2 * run;
        const int ty = fdiv(t, dm.ws, mul_ws), tx = t - ty * dm.ws;
        const int y = y0 + ty, x = x0 + tx;
        float2 acc[2] = {bias2, bias2};
        if (lce) {
            const bool inside = y >= 2 && y + 2 < dm.H && x >= 2 && x + run + 1 < dm.W;
#pragma unroll
            for (int ti = 0; ti < 5; ++ti) {
                const int yy = y + ti - 2;
                float2 v[6];
#pragma unroll
                for (int xx = 0; xx < 6; ++xx) {
                    if (xx < run + 4) {
                        const int xc = x + xx - 2;
                        uint32_t w = 0u;
                        if (inside || ((unsigned)yy < (unsigned)dm.H && (unsigned)xc < (unsigned)dm.W)) {
                            const int tok = yy * dm.W + xc;
                            w = ptx::lds_u32(vbase + tok * 64 + ((cq ^ ((tok >> 1) & 3)) << 4) + vcol);
                        }
                        v[xx] = make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
                    }
                }
#pragma unroll
                for (int tj = 0; tj < 5; ++tj) {
                    acc[0] = __ffma2_rn(wv[ti * 5 + tj], v[tj], acc[0]);
                    if (run == 2) acc[1] = __ffma2_rn(wv[ti * 5 + tj], v[tj + 1], acc[1]);
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            if (e < run) {
                const float2 att = *reinterpret_cast<const float2*>(stage_o + (t - t0 + e) * 32 + 2 * cp);
                const float2 r2 = __fadd2_rn(att, acc[e]);
                outb[((size_t)y * dm.W + x + e) * (dm.C / 2)] = pack2_bf16(r2.x, r2.y);
            }
        }
    }
}


// ---- MMAs against rows gathered from a resident slice.  trow[e]: the row of column lane + 32 e of
// the current block of 64 columns, as its byte offset in the slice with the row's swizzle phase in
// bits 4-5 (img_row_offset); the lane that needs another column's row gets it by shuffle and only
// has to xor in its own 16-byte chunk.  Slices start on 64-byte boundaries.
__device__ __forceinline__ int img_row_offset(int tok) { return tok * 64 + (((tok >> 1) & 3) << 4); }
// C[16 x 64] = A (16 x 32 channels) * rows^T: column c of C is the dot product with row trow(c)
__device__ __forceinline__ void img_rows_x_gather_t(float c[8][4], const uint32_t a[2][4], uint32_t slice,
                                                    const int trow[2], int lane) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint32_t b[4];
        const int xo = __shfl_sync(0xffffffffu, trow[j >> 2], ((8 * j) & 31) + (lane & 7));
        ldmatrix_x4(slice + (xo ^ ((lane >> 3) << 4)), b);        // lane >> 3: channel chunk of this lane's matrix
        mma_bf16_zero(c[j], a[0], b[0], b[1]);
        mma_bf16(c[j], a[1], b[2], b[3]);
    }
}
// acc[16 x 32 channels] += A (16 x 64 columns, four k-step fragments) * rows
__device__ __forceinline__ void img_frag_x_gather(float acc[4][4], const uint32_t a[4][4], uint32_t slice,
                                                  const int trow[2], int lane) {
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int xo = __shfl_sync(0xffffffffu, trow[s >> 1], ((16 * s) & 31) + (lane & 7) + ((lane >> 3) & 1) * 8);
#pragma unroll
        for (int np = 0; np < 2; ++np) {
            uint32_t b[4];
            ldmatrix_x4_trans(slice + (xo ^ ((2 * np + (lane >> 4)) << 4)), b);
            mma_bf16(acc[2 * np], a[s], b[0], b[1]);
            mma_bf16(acc[2 * np + 1], a[s], b[2], b[3]);
        }
    }
}
// The same two products against the rows of TWO slices that share their row numbers (K and V, or Q
// and dO): one shuffle and one address per pair of loads.
__device__ __forceinline__ void img_rows_x_gather_t2(float c1[8][4], const uint32_t a1[2][4], uint32_t slice1,
                                                     float c2[8][4], const uint32_t a2[2][4], uint32_t slice2,
                                                     const int trow[2], int lane) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint32_t b[4];
        const int xo = __shfl_sync(0xffffffffu, trow[j >> 2], ((8 * j) & 31) + (lane & 7)) ^ ((lane >> 3) << 4);
        ldmatrix_x4(slice1 + xo, b);
        mma_bf16_zero(c1[j], a1[0], b[0], b[1]);
        mma_bf16(c1[j], a1[1], b[2], b[3]);
        ldmatrix_x4(slice2 + xo, b);
        mma_bf16_zero(c2[j], a2[0], b[0], b[1]);
        mma_bf16(c2[j], a2[1], b[2], b[3]);
    }
}
__device__ __forceinline__ void img_frag_x_gather2(float acc1[4][4], const uint32_t a1[4][4], uint32_t slice1,
                                                   float acc2[4][4], const uint32_t a2[4][4], uint32_t slice2,
                                                   const int trow[2], int lane) {
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int xo = __shfl_sync(0xffffffffu, trow[s >> 1], ((16 * s) & 31) + (lane & 7) + ((lane >> 3) & 1) * 8);
#pragma unroll
        for (int np = 0; np < 2; ++np) {
            uint32_t b[4];
            const int xq = xo ^ ((2 * np + (lane >> 4)) << 4);
            ldmatrix_x4_trans(slice1 + xq, b);
            mma_bf16(acc1[2 * np], a1[s], b[0], b[1]);
            mma_bf16(acc1[2 * np + 1], a1[s], b[2], b[3]);
            ldmatrix_x4_trans(slice2 + xq, b);
            mma_bf16(acc2[2 * np], a2[s], b[0], b[1]);
            mma_bf16(acc2[2 * np + 1], a2[s], b[2], b[3]);
        }
    }
}
// A fragments (rows g and g + 8 of a 16-token tile of a region, 32 channels) straight from global
// memory; rows beyond `rows` are zero.  base: the image's first token, offset to the head.
__device__ __forceinline__ void img_load_a_global(uint32_t a[2][4], const uint8_t* base, int y0, int x0, int t0,
                                                  int rows, int ws, uint32_t mul_ws, size_t row_bytes,
                                                  size_t tok_bytes, int lane) {
    const int g = lane >> 2, tq = lane & 3;
    const int ta = t0 + g, tb = t0 + g + 8;
    const bool va = g < rows, vb = g + 8 < rows;
    const int tya = fdiv(va ? ta : 0, ws, mul_ws), txa = (va ? ta : 0) - tya * ws;
    const int tyb = fdiv(vb ? tb : 0, ws, mul_ws), txb = (vb ? tb : 0) - tyb * ws;
    const uint8_t* pa = base + (size_t)(y0 + tya) * row_bytes + (size_t)(x0 + txa) * tok_bytes + 4 * tq;
    const uint8_t* pb = base + (size_t)(y0 + tyb) * row_bytes + (size_t)(x0 + txb) * tok_bytes + 4 * tq;
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        a[s][0] = va ? ldg_u32(pa + 32 * s) : 0u;
        a[s][1] = vb ? ldg_u32(pb + 32 * s) : 0u;
        a[s][2] = va ? ldg_u32(pa + 32 * s + 16) : 0u;
        a[s][3] = vb ? ldg_u32(pb + 32 * s + 16) : 0u;
    }
}

// which instantiation a problem takes
inline int img_region_shape(const Dims& d) {
    if (d.ws == 4 && d.hs == 4) return 44;
    if (d.ws == 2 && d.hs == 2) return 22;
    return 0;
}

}  // namespace bra
