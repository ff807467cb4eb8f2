// Gradients of the routed attention for a fixed routing index (Eq. 7 with Eq. 1) with
// warp-level tensor-core MMAs: head dim 32, bf16, any region shape and any topk.
// With P the softmax of Eq. 1 over a group's routed keys (recomputed from the saved
// log-sum-exp): dP = dO V^g^T, delta = rowsum(P o dP), dS = P o (dP - delta),
//   dQ = scale dS K^g                                    (query-centric kernel)
//   dK_j = scale sum dS^T Q, dV_j = sum P^T dO  over the query regions that routed to j,
//   in the fixed order of the inverse routing index      (key-centric kernel)
//   dV += LCE adjoint of dO (5x5 depthwise correlation with the flipped filter).
// Both kernels mirror the forward warp-level kernel: one warp = 16 rows, the other side
// streamed in blocks of 64 through shared memory, S / P / dP / dS in registers.  No atomics:
// every sum has a fixed order, results are bit-identical from run to run.
#include "mma_common.cuh"

namespace bra {

using namespace ptx;

struct BwdGeom {
    MmaGeom g;
    int off_a2;        // second row operand (dO rows in the dQ kernel, V rows in the dK/dV kernel)
    int off_stat;      // per-column lse * log2(e) and delta: [stages][2][64] floats (dK/dV kernel)
    int smem_bytes;
};

// one row = one token's 64 bytes of a head = 4 chunks of 16 B, chunk index xor (row >> 1) & 3
__device__ __forceinline__ void load_row64(uint32_t dst_row, int row, const uint8_t* src, const uint8_t* safe, bool valid) {
    const uint32_t sw = (row >> 1) & 3;
#pragma unroll
    for (int q = 0; q < 4; ++q)
        cp_async_16(dst_row + ((q ^ sw) << 4), valid ? src + q * 16 : safe, valid ? 16u : 0u);
}
// A fragments (16 rows x 32 channels, two k-steps) of rows [16 * warp, +16) of a row tile
__device__ __forceinline__ void load_a_frags(uint32_t tile, int warp, int lane, uint32_t a[2][4]) {
    const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        const int q = 2 * s + (lane >> 4);
        ldmatrix_x4(tile + row * 64 + ((q ^ ((row >> 1) & 3)) << 4), a[s]);
    }
}
// C[16 x 64] = A (16 x 32) * B^T where B is a [64 rows][32 channels] tile (rows = columns of C)
__device__ __forceinline__ void mma_rows_x_tile_t(float c[8][4], const uint32_t a[2][4], uint32_t tile, int lane) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        c[j][0] = c[j][1] = c[j][2] = c[j][3] = 0.f;
        uint32_t b[4];
        const int r = 8 * j + (lane & 7);
        const int q = lane >> 3;
        ldmatrix_x4(tile + r * 64 + ((q ^ ((r >> 1) & 3)) << 4), b);
        mma_bf16(c[j], a[0], b[0], b[1]);
        mma_bf16(c[j], a[1], b[2], b[3]);
    }
}
// acc[16 x 32] += A (16 x 64, as four k-step fragments) * B where B is a [64 rows][32 channels] tile
__device__ __forceinline__ void mma_frag_x_tile(float acc[4][4], const uint32_t a[4][4], uint32_t tile, int lane) {
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int r = 16 * s + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int np = 0; np < 2; ++np) {
            uint32_t b[4];
            const int q = 2 * np + (lane >> 4);
            ldmatrix_x4_trans(tile + r * 64 + ((q ^ ((r >> 1) & 3)) << 4), b);
            mma_bf16(acc[2 * np], a[s], b[0], b[1]);
            mma_bf16(acc[2 * np + 1], a[s], b[2], b[3]);
        }
    }
}

// ------------------------------------------------------------------ dQ and delta
__global__ void __launch_bounds__(wm::MAXW * 32)
bwd_dq_mma_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                  const __nv_bfloat16* __restrict__ Vg, const int32_t* __restrict__ index,
                  const float* __restrict__ lse, const __nv_bfloat16* __restrict__ dOg,
                  __nv_bfloat16* __restrict__ dQg, float* __restrict__ delta_out,
                  int32_t* __restrict__ status, Dims dm, BwdGeom bg) {
    using namespace wm;
    const MmaGeom& gm = bg.g;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = gm.nw * 32;

    int bid = blockIdx.x;
    const int ck = bid % gm.chunks; bid /= gm.chunks;
    const int h = bid % dm.heads; bid /= dm.heads;
    const int i = bid % dm.R;
    const int b = bid / dm.R;
    const int t0 = ck * gm.nw * 16;
    const int ry = fdiv(i, dm.S, gm.mul_s), rx = i - ry * dm.S;
    const int y0 = ry * dm.hs, x0 = rx * dm.ws;
    const size_t tok_bytes = (size_t)dm.C * 2;
    const size_t row_bytes = (size_t)dm.W * tok_bytes;
    const size_t img = (size_t)b * dm.H * row_bytes;
    const size_t ch_off = (size_t)h * 64;
    const uint8_t* Qb = reinterpret_cast<const uint8_t*>(Qg) + img + ch_off;
    const uint8_t* Kb = reinterpret_cast<const uint8_t*>(Kg) + img + ch_off;
    const uint8_t* Vb = reinterpret_cast<const uint8_t*>(Vg) + img + ch_off;
    const uint8_t* Gb = reinterpret_cast<const uint8_t*>(dOg) + img + ch_off;
    const int hi = dm.heads_i == 1 ? 0 : h;
    const int32_t* irow = index + (((size_t)b * dm.heads_i + hi) * dm.R + i) * dm.topk;
    const int total_keys = dm.topk * dm.n_r;
    const size_t stat0 = ((size_t)b * dm.heads + h) * dm.N;

    int32_t* s_idx = reinterpret_cast<int32_t*>(smem + gm.off_idx);
    uint8_t* s_flag = smem + gm.off_flag;
    for (int m = tid; m < dm.topk; m += nthreads) {
        int r = __ldg(irow + m);
        if (r < 0 || r >= dm.R) { record_error(status, BRA_ERR_INDEX, r); r = -1; }
        s_idx[m] = r;
    }
    __syncthreads();

    auto load_kv_block = [&](int blk, int stage) {
        const uint32_t kdst = sbase + gm.off_kv + stage * 8192, vdst = kdst + 4096;
        for (int key = tid; key < KB; key += nthreads) {
            const int kk = blk * KB + key;
            bool valid = kk < total_keys;
            size_t off = 0;
            if (valid) {
                const int m = fdiv(kk, dm.n_r, gm.mul_nr), t = kk - m * dm.n_r;
                const int r = s_idx[m];
                valid = r >= 0;
                if (valid) {
                    const int qy = fdiv(r, dm.S, gm.mul_s), qx = r - qy * dm.S;
                    const int ty = fdiv(t, dm.ws, gm.mul_ws), tx = t - ty * dm.ws;
                    off = (size_t)(qy * dm.hs + ty) * row_bytes + (size_t)(qx * dm.ws + tx) * tok_bytes;
                }
            }
            s_flag[stage * KB + key] = valid ? 1 : 0;
            load_row64(kdst + key * 64, key, Kb + off, Kb, valid);
            load_row64(vdst + key * 64, key, Vb + off, Kb, valid);
        }
    };
    for (int row = tid; row < gm.nw * 16; row += nthreads) {
        const int t = t0 + row;
        const bool valid = t < dm.n_r;
        const int ty = fdiv(valid ? t : 0, dm.ws, gm.mul_ws), tx = (valid ? t : 0) - ty * dm.ws;
        const size_t off = (size_t)(y0 + ty) * row_bytes + (size_t)(x0 + tx) * tok_bytes;
        load_row64(sbase + gm.off_q + row * 64, row, Qb + off, Kb, valid);
        load_row64(sbase + bg.off_a2 + row * 64, row, Gb + off, Kb, valid);
    }
    load_kv_block(0, 0);
    cp_async_commit();

    const int g = lane >> 2, tq = lane & 3;
    const float sl2 = dm.scale * 1.4426950408889634f;
    // rows g and g + 8 of this warp: token, statistics
    int tok[2]; bool rvalid[2]; float lse2[2]; size_t spos[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        tok[r] = t0 + warp * 16 + g + 8 * r;
        rvalid[r] = tok[r] < dm.n_r;
        const int t = rvalid[r] ? tok[r] : 0;
        const int ty = fdiv(t, dm.ws, gm.mul_ws), tx = t - ty * dm.ws;
        spos[r] = (size_t)(y0 + ty) * dm.W + x0 + tx;
        lse2[r] = rvalid[r] ? __ldg(lse + stat0 + spos[r]) * 1.4426950408889634f : 0.f;
    }
    float delta[2] = {0.f, 0.f};
    float dq[4][4];
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) dq[n][e] = 0.f;
    uint32_t qa[2][4], ga[2][4];

    const bool single = gm.nblocks == 1;          // S, P, dP of the only block stay in registers
    const int iters = single ? 1 : 2 * gm.nblocks; // otherwise: one sweep for delta, one for dQ
    for (int it = 0; it < iters; ++it) {
        const int blk = it % gm.nblocks, sweep = it / gm.nblocks;
        const int stage = gm.stages == 2 ? (it & 1) : 0;
        if (gm.stages == 2 && it + 1 < iters) {
            load_kv_block((it + 1) % gm.nblocks, stage ^ 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (it == 0) {
            load_a_frags(sbase + gm.off_q, warp, lane, qa);
            load_a_frags(sbase + bg.off_a2, warp, lane, ga);
        }
        const uint32_t kbase = sbase + gm.off_kv + stage * 8192, vbase = kbase + 4096;
        float c[8][4], dp[8][4];
        mma_rows_x_tile_t(c, qa, kbase, lane);       // S = Q K^T
        mma_rows_x_tile_t(dp, ga, vbase, lane);      // dP = dO V^T
        const uint8_t* fl = s_flag + stage * KB;
        // P = exp(S scale - lse); keys that do not count give 0
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uchar2 f = *reinterpret_cast<const uchar2*>(fl + 8 * j + 2 * tq);
            c[j][0] = f.x ? ex2_approx(fmaf(c[j][0], sl2, -lse2[0])) : 0.f;
            c[j][1] = f.y ? ex2_approx(fmaf(c[j][1], sl2, -lse2[0])) : 0.f;
            c[j][2] = f.x ? ex2_approx(fmaf(c[j][2], sl2, -lse2[1])) : 0.f;
            c[j][3] = f.y ? ex2_approx(fmaf(c[j][3], sl2, -lse2[1])) : 0.f;
        }
        if (sweep == 0) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                delta[0] = fmaf(c[j][0], dp[j][0], fmaf(c[j][1], dp[j][1], delta[0]));
                delta[1] = fmaf(c[j][2], dp[j][2], fmaf(c[j][3], dp[j][3], delta[1]));
            }
            if (single || blk == gm.nblocks - 1) {
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    delta[r] += __shfl_xor_sync(0xffffffffu, delta[r], 1);
                    delta[r] += __shfl_xor_sync(0xffffffffu, delta[r], 2);
                }
            }
        }
        if (single || sweep == 1) {
            uint32_t sa[4][4];                       // dS as A fragments
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                sa[j >> 1][(j & 1) * 2] = pack2_bf16(c[j][0] * (dp[j][0] - delta[0]), c[j][1] * (dp[j][1] - delta[0]));
                sa[j >> 1][(j & 1) * 2 + 1] = pack2_bf16(c[j][2] * (dp[j][2] - delta[1]), c[j][3] * (dp[j][3] - delta[1]));
            }
            mma_frag_x_tile(dq, sa, kbase, lane);    // dQ += dS K
        }
        __syncthreads();
    }

    // ---- dQ = scale * acc, delta kept for the dK/dV kernel ----
    uint32_t* out = reinterpret_cast<uint32_t*>(dQg) + (img + ch_off) / 4 + tq;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        if (!rvalid[r]) continue;
        uint32_t* o = out + spos[r] * (dm.C / 2);
#pragma unroll
        for (int n = 0; n < 4; ++n)
            o[4 * n] = pack2_bf16(dq[n][2 * r] * dm.scale, dq[n][2 * r + 1] * dm.scale);
        if (tq == 0) delta_out[stat0 + spos[r]] = delta[r];
    }
}

// ------------------------------------------------------------------ dK, dV
__global__ void __launch_bounds__(wm::MAXW * 32)
bwd_dkv_mma_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                   const __nv_bfloat16* __restrict__ Vg, const int32_t* __restrict__ inv_off,
                   const int32_t* __restrict__ inv_list, const float* __restrict__ lse,
                   const float* __restrict__ delta, const __nv_bfloat16* __restrict__ dOg,
                   const float* __restrict__ lce_w, __nv_bfloat16* __restrict__ dKg,
                   __nv_bfloat16* __restrict__ dVg, Dims dm, BwdGeom bg) {
    using namespace wm;
    const MmaGeom& gm = bg.g;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = gm.nw * 32;

    int bid = blockIdx.x;
    const int ck = bid % gm.chunks; bid /= gm.chunks;
    const int h = bid % dm.heads; bid /= dm.heads;
    const int jr = bid % dm.R;                       // key region
    const int b = bid / dm.R;
    const int t0 = ck * gm.nw * 16;
    const int t1 = min(dm.n_r, t0 + gm.nw * 16);
    const int ry = fdiv(jr, dm.S, gm.mul_s), rx = jr - ry * dm.S;
    const int y0 = ry * dm.hs, x0 = rx * dm.ws;
    const size_t tok_bytes = (size_t)dm.C * 2;
    const size_t row_bytes = (size_t)dm.W * tok_bytes;
    const size_t img = (size_t)b * dm.H * row_bytes;
    const size_t ch_off = (size_t)h * 64;
    const uint8_t* Qb = reinterpret_cast<const uint8_t*>(Qg) + img + ch_off;
    const uint8_t* Kb = reinterpret_cast<const uint8_t*>(Kg) + img + ch_off;
    const uint8_t* Vb = reinterpret_cast<const uint8_t*>(Vg) + img + ch_off;
    const uint8_t* Gb = reinterpret_cast<const uint8_t*>(dOg) + img + ch_off;
    const int hi = dm.heads_i == 1 ? 0 : h;
    const size_t bh = (size_t)b * dm.heads_i + hi;
    const int e0 = __ldg(inv_off + bh * (dm.R + 1) + jr), e1 = __ldg(inv_off + bh * (dm.R + 1) + jr + 1);
    const int32_t* list = inv_list + bh * dm.R * dm.topk + e0;   // query regions that list jr, fixed order
    const int total_cols = (e1 - e0) * dm.n_r;
    const int nblocks = (total_cols + KB - 1) / KB;
    const size_t stat0 = ((size_t)b * dm.heads + h) * dm.N;
    uint8_t* s_flag = smem + gm.off_flag;
    float* s_stat = reinterpret_cast<float*>(smem + bg.off_stat);

    // column block: queries of the listed regions, 64 at a time: Q rows, dO rows, lse, delta
    auto load_col_block = [&](int blk, int stage) {
        const uint32_t qdst = sbase + gm.off_kv + stage * 8192, gdst = qdst + 4096;
        for (int col = tid; col < KB; col += nthreads) {
            const int cc = blk * KB + col;
            const bool valid = cc < total_cols;
            size_t off = 0, sp = 0;
            if (valid) {
                const int m = fdiv(cc, dm.n_r, gm.mul_nr), t = cc - m * dm.n_r;
                const int r = __ldg(list + m);
                const int qy = fdiv(r, dm.S, gm.mul_s), qx = r - qy * dm.S;
                const int ty = fdiv(t, dm.ws, gm.mul_ws), tx = t - ty * dm.ws;
                off = (size_t)(qy * dm.hs + ty) * row_bytes + (size_t)(qx * dm.ws + tx) * tok_bytes;
                sp = (size_t)(qy * dm.hs + ty) * dm.W + qx * dm.ws + tx;
            }
            s_flag[stage * KB + col] = valid ? 1 : 0;
            s_stat[stage * 128 + col] = valid ? __ldg(lse + stat0 + sp) * 1.4426950408889634f : 0.f;
            s_stat[stage * 128 + 64 + col] = valid ? __ldg(delta + stat0 + sp) : 0.f;
            load_row64(qdst + col * 64, col, Qb + off, Kb, valid);
            load_row64(gdst + col * 64, col, Gb + off, Kb, valid);
        }
    };
    // K and V rows of this chunk of the key region
    for (int row = tid; row < gm.nw * 16; row += nthreads) {
        const int t = t0 + row;
        const bool valid = t < dm.n_r;
        const int ty = fdiv(valid ? t : 0, dm.ws, gm.mul_ws), tx = (valid ? t : 0) - ty * dm.ws;
        const size_t off = (size_t)(y0 + ty) * row_bytes + (size_t)(x0 + tx) * tok_bytes;
        load_row64(sbase + gm.off_q + row * 64, row, Kb + off, Kb, valid);
        load_row64(sbase + bg.off_a2 + row * 64, row, Vb + off, Kb, valid);
    }
    // dO halo of the chunk's token rows for the LCE adjoint
    const int cy0 = fdiv(t0, dm.ws, gm.mul_ws);
    const int cy1 = fdiv(t1 - 1, dm.ws, gm.mul_ws);
    const int hrows = cy1 - cy0 + 5;
    if (dm.lce) {
        const int cells = hrows * gm.halo_w;
        for (int cell = tid; cell < cells; cell += nthreads) {
            const int hy = cell / gm.halo_w, hx = cell - hy * gm.halo_w;
            const int y = y0 + cy0 + hy - 2, x = x0 + hx - 2;
            const bool valid = (unsigned)y < (unsigned)dm.H && (unsigned)x < (unsigned)dm.W;
            const uint8_t* src = Gb + (size_t)(valid ? y : 0) * row_bytes + (size_t)(valid ? x : 0) * tok_bytes;
            const uint32_t dst = sbase + gm.off_halo + cell * 64;
#pragma unroll
            for (int q = 0; q < 4; ++q) cp_async_16(dst + q * 16, valid ? src + q * 16 : Kb, valid ? 16u : 0u);
        }
    }
    if (nblocks > 0) load_col_block(0, 0);
    cp_async_commit();

    const int g = lane >> 2, tq = lane & 3;
    const float sl2 = dm.scale * 1.4426950408889634f;
    float dk[4][4], dv[4][4];
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) { dk[n][e] = 0.f; dv[n][e] = 0.f; }
    uint32_t ka[2][4], va[2][4];

    for (int blk = 0; blk < nblocks; ++blk) {
        const int stage = blk & 1;
        if (blk + 1 < nblocks) {
            load_col_block(blk + 1, stage ^ 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (blk == 0) {
            load_a_frags(sbase + gm.off_q, warp, lane, ka);
            load_a_frags(sbase + bg.off_a2, warp, lane, va);
        }
        const uint32_t qbase = sbase + gm.off_kv + stage * 8192, gbase = qbase + 4096;
        float c[8][4], dp[8][4];
        mma_rows_x_tile_t(c, ka, qbase, lane);       // S^T = K Q^T
        mma_rows_x_tile_t(dp, va, gbase, lane);      // dP^T = V dO^T
        const uint8_t* fl = s_flag + stage * KB;
        const float* st = s_stat + stage * 128;
        uint32_t pa[4][4], sa[4][4];                 // P^T and dS^T as A fragments
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int col = 8 * j + 2 * tq;
            const uchar2 f = *reinterpret_cast<const uchar2*>(fl + col);
            const float2 l2 = *reinterpret_cast<const float2*>(st + col);
            const float2 dl = *reinterpret_cast<const float2*>(st + 64 + col);
            const float p0 = f.x ? ex2_approx(fmaf(c[j][0], sl2, -l2.x)) : 0.f;
            const float p1 = f.y ? ex2_approx(fmaf(c[j][1], sl2, -l2.y)) : 0.f;
            const float p2 = f.x ? ex2_approx(fmaf(c[j][2], sl2, -l2.x)) : 0.f;
            const float p3 = f.y ? ex2_approx(fmaf(c[j][3], sl2, -l2.y)) : 0.f;
            pa[j >> 1][(j & 1) * 2] = pack2_bf16(p0, p1);
            pa[j >> 1][(j & 1) * 2 + 1] = pack2_bf16(p2, p3);
            sa[j >> 1][(j & 1) * 2] = pack2_bf16(p0 * (dp[j][0] - dl.x), p1 * (dp[j][1] - dl.y));
            sa[j >> 1][(j & 1) * 2 + 1] = pack2_bf16(p2 * (dp[j][2] - dl.x), p3 * (dp[j][3] - dl.y));
        }
        mma_frag_x_tile(dk, sa, qbase, lane);        // dK += dS^T Q
        mma_frag_x_tile(dv, pa, gbase, lane);        // dV += P^T dO
        __syncthreads();
    }
    if (nblocks == 0) {
        cp_async_wait<0>();
        __syncthreads();
    }

    // ---- dK = scale * acc; dV staged fp32 [token][32 ch] over the column buffers ----
    float* stage_v = reinterpret_cast<float*>(smem + gm.off_kv);
    uint32_t* outk = reinterpret_cast<uint32_t*>(dKg) + (img + ch_off) / 4 + tq;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = warp * 16 + g + 8 * r;
        const int t = t0 + row;
        if (t < dm.n_r) {
            const int ty = fdiv(t, dm.ws, gm.mul_ws), tx = t - ty * dm.ws;
            uint32_t* o = outk + ((size_t)(y0 + ty) * dm.W + x0 + tx) * (dm.C / 2);
#pragma unroll
            for (int n = 0; n < 4; ++n) {
                o[4 * n] = pack2_bf16(dk[n][2 * r] * dm.scale, dk[n][2 * r + 1] * dm.scale);
                *reinterpret_cast<float2*>(stage_v + row * 32 + 8 * n + 2 * tq) = make_float2(dv[n][2 * r], dv[n][2 * r + 1]);
            }
        }
    }
    __syncthreads();

    // ---- LCE adjoint + store of dV: dV[y,x] += sum_ij w[i,j] dO[y-i+2, x-j+2] = correlation with the flipped filter ----
    {
        const int cp = tid & 15;
        const int run = (dm.ws & 1) ? 1 : 2;
        const int nruns = (t1 - t0) / run;
        float2 wv[25];
        if (dm.lce) {
            const float* wp = lce_w + (size_t)(h * 32 + 2 * cp) * 25;
#pragma unroll
            for (int q = 0; q < 25; ++q) wv[q] = make_float2(__ldg(wp + 24 - q), __ldg(wp + 25 + 24 - q));
        }
        const uint32_t halo = sbase + gm.off_halo + cp * 4;
        uint32_t* out = reinterpret_cast<uint32_t*>(dVg) + (img + ch_off) / 4 + cp;
        for (int u = tid >> 4; u < nruns; u += nthreads >> 4) {
            const int t = t0 + u * run;
            const int ty = fdiv(t, dm.ws, gm.mul_ws), tx = t - ty * dm.ws;
            float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            if (dm.lce) {
#pragma unroll
                for (int ti = 0; ti < 5; ++ti) {
                    const uint32_t hrow = halo + ((ty - cy0 + ti) * gm.halo_w + tx) * 64;
                    float2 v[6];
#pragma unroll
                    for (int xx = 0; xx < 6; ++xx) {
                        if (xx < run + 4) {
                            const uint32_t w = lds_u32(hrow + xx * 64);
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
                    const float2 a = *reinterpret_cast<const float2*>(stage_v + (t - t0 + e) * 32 + 2 * cp);
                    const float2 r2 = __fadd2_rn(a, acc[e]);
                    out[((size_t)(y0 + ty) * dm.W + x0 + tx + e) * (dm.C / 2)] = pack2_bf16(r2.x, r2.y);
                }
            }
        }
    }
}

// ------------------------------------------------------------------ host side
static BwdGeom bwd_geom(const Dims& d, bool key_centric) {
    BwdGeom bg;
    bg.g = mma_geom(d);
    MmaGeom& g = bg.g;
    if (key_centric) g.stages = 2;                 // the number of column blocks is only known on the device
    int off = 0;
    g.off_q = off;     off += g.nw * 16 * 64;
    bg.off_a2 = off;   off += g.nw * 16 * 64;
    g.off_kv = off;    off += g.stages * 8192;      // dK/dV kernel: also the fp32 staging tile of dV
    g.off_flag = off;  off += g.stages * wm::KB;
    off = (off + 15) / 16 * 16;
    bg.off_stat = off; off += key_centric ? g.stages * 128 * 4 : 0;
    g.off_idx = off;   off += key_centric ? 0 : ((d.topk * 4 + 15) / 16) * 16;
    g.off_halo = off;  off += (key_centric && d.lce) ? g.halo_rows * g.halo_w * 64 : 0;
    bg.smem_bytes = off;
    return bg;
}

bool backward_mma_supported(const Dims& d, int dtype) {
    if (d.d != 32 || !attend_mma_supported(d, dtype)) return false;      // the gradient kernels are built for head dim 32
    const BwdGeom a = bwd_geom(d, false), b = bwd_geom(d, true);
    return a.smem_bytes <= 200 * 1024 && b.smem_bytes <= 200 * 1024 && b.g.nw * 2048 <= b.g.stages * 8192;
}

cudaError_t launch_backward_mma(const Dims& d, const void* Q, const void* K, const void* V,
                                const int32_t* index, const int32_t* inv_off, const int32_t* inv_list,
                                const float* lce_w, const float* lse, const void* dO,
                                void* dQ, void* dK, void* dV, float* delta, int32_t* status, cudaStream_t st) {
    const BwdGeom a = bwd_geom(d, false), b = bwd_geom(d, true);
    static PerDeviceMax smem_a, smem_b;
    cudaError_t e;
    if (a.smem_bytes > 48 * 1024 &&
        (e = smem_a.ensure(a.smem_bytes, [&] {
             return cudaFuncSetAttribute(bwd_dq_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, a.smem_bytes);
         })) != cudaSuccess)
        return e;
    if (b.smem_bytes > 48 * 1024 &&
        (e = smem_b.ensure(b.smem_bytes, [&] {
             return cudaFuncSetAttribute(bwd_dkv_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, b.smem_bytes);
         })) != cudaSuccess)
        return e;
    const unsigned grid = (unsigned)((long long)d.B * d.R * d.heads * a.g.chunks);
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(Q);
    const __nv_bfloat16* k = static_cast<const __nv_bfloat16*>(K);
    const __nv_bfloat16* v = static_cast<const __nv_bfloat16*>(V);
    const __nv_bfloat16* go = static_cast<const __nv_bfloat16*>(dO);
    bwd_dq_mma_kernel<<<grid, a.g.nw * 32, a.smem_bytes, st>>>(q, k, v, index, lse, go, static_cast<__nv_bfloat16*>(dQ),
                                                             delta, status, d, a);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    bwd_dkv_mma_kernel<<<grid, b.g.nw * 32, b.smem_bytes, st>>>(q, k, v, inv_off, inv_list, lse, delta, go, lce_w,
                                                              static_cast<__nv_bfloat16*>(dK),
                                                              static_cast<__nv_bfloat16*>(dV), d, b);
    count_launch();
    return cudaGetLastError();
}

}  // namespace bra
