// Routed token-to-token attention + LCE with warp-level tensor-core MMAs
// (Eq. 6, Eq. 7 with Eq. 1): head dim 32 or 64, bf16, any region shape and any topk.
//
// tcgen05 MMAs work on 128-row tiles; a BRA query group is one region's n_r tokens of one
// head, each group with its own routed keys, so for small regions (n_r = 4 or 16) a 128-row
// tile would be 8-32x padding.  The warp-level m16n8k16 MMA has the matching granularity:
// one warp = 16 query rows of one (image, region, head), streaming that group's routed keys
// in blocks of 64, flash-attention style, with S, P and O in registers.
//
// CTA = (image b, query region i, head h, chunk of up to 128 of the region's tokens):
//   1. all threads: cp.async the Q rows, the V halo of the chunk and, block by block
//      (double-buffered), the K and V rows of the routed regions: K^g / V^g are never
//      formed in HBM, the routing index only picks source addresses.  Rows are 64 bytes
//      (this head's 32 channels) with a 16-byte-chunk xor swizzle for ldmatrix.
//   2. per warp and key block: S = Q K^T (16 MMAs), online softmax on the fragments
//      (quad shuffles), O += P V (16 MMAs).
//   3. normalised O^att to an fp32 staging tile (over the dead K/V buffers).
//   4. all threads: LCE from the halo tile (thread = channel pair x run of 2 tokens),
//      + O^att, bf16 store of O.
// A head of 64 channels (template parameter PL = 2) is handled as two planes of 32: every tile
// (Q, K, V, halo, staging) exists once per plane in the layout above, S sums the two planes'
// products, O and the LCE run per plane.
#include "mma_common.cuh"

namespace bra {

using namespace ptx;

template <int PL>
__global__ void __launch_bounds__(wm::MAXW * 32)
attend_mma_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                  const __nv_bfloat16* __restrict__ Vg, const int32_t* index,
                  const float* __restrict__ lce_w, const float* __restrict__ lce_b,
                  __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
                  int32_t* __restrict__ status, Dims dm, MmaGeom gm) {
    using namespace wm;
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = gm.nw * 32;
    pdl_wait();          // in bra_forward the launch may overlap the tail of the routing kernel

    // ---- which group and chunk ----
    int bid = blockIdx.x;
    const int ck = bid % gm.chunks; bid /= gm.chunks;
    const int h = bid % dm.heads; bid /= dm.heads;
    const int i = bid % dm.R;
    const int b = bid / dm.R;
    const int t0 = ck * gm.nw * 16;                                   // first token of the chunk (raster in region)
    const int t1 = min(dm.n_r, t0 + gm.nw * 16);
    const int ry = fdiv(i, dm.S, gm.mul_s), rx = i - ry * dm.S;
    const int y0 = ry * dm.hs, x0 = rx * dm.ws;                       // region origin in the map
    const size_t tok_bytes = (size_t)dm.C * 2;
    const size_t row_bytes = (size_t)dm.W * tok_bytes;
    const size_t img = (size_t)b * dm.H * row_bytes;
    const size_t ch_off = (size_t)h * 64 * PL;                        // this head's 32 * PL channels
    const uint8_t* Qb = reinterpret_cast<const uint8_t*>(Qg) + img + ch_off;
    const uint8_t* Kb = reinterpret_cast<const uint8_t*>(Kg) + img + ch_off;
    const uint8_t* Vb = reinterpret_cast<const uint8_t*>(Vg) + img + ch_off;
    const int hi = dm.heads_i == 1 ? 0 : h;
    const int32_t* irow = index + (((size_t)b * dm.heads_i + hi) * dm.R + i) * dm.topk;
    const int total_keys = dm.topk * dm.n_r;

    int32_t* s_idx = reinterpret_cast<int32_t*>(smem + gm.off_idx);
    uint8_t* s_flag = smem + gm.off_flag;                             // [stages][64]: 1 = key counts
    // ---- routing entries of this group: region origin per slot, -1 if out of range ----
    for (int m = tid; m < dm.topk; m += nthreads) {
        int r = __ldcg(irow + m);   // coherent load: the index may come from the kernel this one overlaps
        if (r < 0 || r >= dm.R) { record_error(status, BRA_ERR_INDEX, r); r = -1; }
        s_idx[m] = r;
    }
    __syncthreads();

    // ---- loaders ----
    // one row = one token's 64 bytes of this head = 4 chunks of 16 B, chunk index xor (row >> 1) & 3
    // (per plane: the next 64 bytes of the token, `plane_bytes` further on in shared memory)
    auto load_row = [&](uint32_t dst_row, int row, const uint8_t* src, bool valid, uint32_t plane_bytes) {
        const uint32_t sw = (row >> 1) & 3;
#pragma unroll
        for (int p = 0; p < PL; ++p)
#pragma unroll
            for (int q = 0; q < 4; ++q)
                cp_async_16(dst_row + p * plane_bytes + ((q ^ sw) << 4), valid ? src + p * 64 + q * 16 : Kb, valid ? 16u : 0u);
    };
    auto load_kv_block = [&](int blk, int stage) {
        const uint32_t kdst = sbase + gm.off_kv + stage * (8192 * PL), vdst = kdst + 4096 * PL;
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
            load_row(kdst + key * 64, key, Kb + off, valid, 4096);
            load_row(vdst + key * 64, key, Vb + off, valid, 4096);
        }
    };
    // Q rows of the chunk (rows beyond the region are zero)
    for (int row = tid; row < gm.nw * 16; row += nthreads) {
        const int t = t0 + row;
        const bool valid = t < dm.n_r;
        const int ty = fdiv(valid ? t : 0, dm.ws, gm.mul_ws), tx = (valid ? t : 0) - ty * dm.ws;
        load_row(sbase + gm.off_q + row * 64, row, Qb + (size_t)(y0 + ty) * row_bytes + (size_t)(x0 + tx) * tok_bytes, valid,
                 gm.nw * 16 * 64);
    }
    // V halo of the chunk's token rows: [rows + 4][ws + 4] tokens x 64 B, zeros outside the map
    const int cy0 = fdiv(t0, dm.ws, gm.mul_ws);                       // first / last region row of the chunk
    const int cy1 = fdiv(t1 - 1, dm.ws, gm.mul_ws);
    const int hrows = cy1 - cy0 + 5;
    if (dm.lce) {
        const int cells = hrows * gm.halo_w;
        for (int cell = tid; cell < cells; cell += nthreads) {
            const int hy = cell / gm.halo_w, hx = cell - hy * gm.halo_w;
            const int y = y0 + cy0 + hy - 2, x = x0 + hx - 2;
            const bool valid = (unsigned)y < (unsigned)dm.H && (unsigned)x < (unsigned)dm.W;
            const uint8_t* src = Vb + (size_t)(valid ? y : 0) * row_bytes + (size_t)(valid ? x : 0) * tok_bytes;
            const uint32_t dst = sbase + gm.off_halo + cell * 64;
#pragma unroll
            for (int p = 0; p < PL; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    cp_async_16(dst + p * (gm.halo_rows * gm.halo_w * 64) + q * 16, valid ? src + p * 64 + q * 16 : Vb, valid ? 16u : 0u);
        }
    }
    load_kv_block(0, 0);
    cp_async_commit();

    // ---- attention: warp = 16 query rows ----
    const int g = lane >> 2, tq = lane & 3;                           // fragment row / column pair
    const float sl2 = dm.scale * 1.4426950408889634f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[PL][4][4];
#pragma unroll
    for (int p = 0; p < PL; ++p)
#pragma unroll
        for (int n = 0; n < 4; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[p][n][e] = 0.f;
    uint32_t qa[PL][2][4];
    const bool lower_only = (t1 - t0) - warp * 16 <= 8;               // rows g + 8 of this warp are padding

    for (int blk = 0; blk < gm.nblocks; ++blk) {
        const int stage = gm.stages == 2 ? (blk & 1) : 0;
        if (gm.stages == 2 && blk + 1 < gm.nblocks) {
            load_kv_block(blk + 1, stage ^ 1);                        // its previous reader finished last iteration
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (blk == 0) {
            // A fragments of Q: ldmatrix x4 per k-step: (rows 0-7, ch lo), (rows 8-15, ch lo), (rows 0-7, ch hi), (rows 8-15, ch hi)
            const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
            for (int p = 0; p < PL; ++p)
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    const int q = 2 * s + (lane >> 4);
                    ldmatrix_x4(sbase + gm.off_q + p * (gm.nw * 16 * 64) + row * 64 + ((q ^ ((row >> 1) & 3)) << 4), qa[p][s]);
                }
        }
        const uint32_t kbase = sbase + gm.off_kv + stage * (8192 * PL), vbase = kbase + 4096 * PL;
        // S = Q K^T: 8 key tiles of 8
        float c[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            c[j][0] = c[j][1] = c[j][2] = c[j][3] = 0.f;
            const int key = 8 * j + (lane & 7);
            const int q = lane >> 3;                                  // channel chunk of this lane's matrix
#pragma unroll
            for (int p = 0; p < PL; ++p) {
                uint32_t kb[4];
                ldmatrix_x4(kbase + p * 4096 + key * 64 + ((q ^ ((key >> 1) & 3)) << 4), kb);
                mma_bf16(c[j], qa[p][0], kb[0], kb[1]);
                mma_bf16(c[j], qa[p][1], kb[2], kb[3]);
            }
        }
        // keys that do not count (padding of the last block, out-of-range entries): -inf
        const uint8_t* fl = s_flag + stage * KB;
        bool all_valid = true;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uchar2 f = *reinterpret_cast<const uchar2*>(fl + 8 * j + 2 * tq);
            if (!f.x) { c[j][0] = -INFINITY; c[j][2] = -INFINITY; all_valid = false; }
            if (!f.y) { c[j][1] = -INFINITY; c[j][3] = -INFINITY; all_valid = false; }
        }
        (void)all_valid;
        // online softmax on rows g (elements 0, 1) and g + 8 (elements 2, 3)
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            mx[0] = fmax3(mx[0], c[j][0], c[j][1]);
            mx[1] = fmax3(mx[1], c[j][2], c[j][3]);
        }
        float corr[2], mneg[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float mnew = fmaxf(m_run[r], mx[r] * sl2);          // sl2 > 0
            corr[r] = (mnew == -INFINITY) ? 1.f : ex2_approx(m_run[r] - mnew);
            mneg[r] = (mnew == -INFINITY) ? 0.f : -mnew;
            m_run[r] = mnew;
            l_run[r] *= corr[r];
        }
#pragma unroll
        for (int p = 0; p < PL; ++p)
#pragma unroll
            for (int n = 0; n < 4; ++n) { o[p][n][0] *= corr[0]; o[p][n][1] *= corr[0]; o[p][n][2] *= corr[1]; o[p][n][3] *= corr[1]; }
        uint32_t pa[4][4];                                            // P as A fragments: 4 k-steps of 16 keys
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float p0 = ex2_approx(fmaf(c[j][0], sl2, mneg[0]));
            const float p1 = ex2_approx(fmaf(c[j][1], sl2, mneg[0]));
            float p2 = 0.f, p3 = 0.f;
            if (!lower_only) {
                p2 = ex2_approx(fmaf(c[j][2], sl2, mneg[1]));
                p3 = ex2_approx(fmaf(c[j][3], sl2, mneg[1]));
            }
            l_run[0] += p0 + p1;
            l_run[1] += p2 + p3;
            pa[j >> 1][(j & 1) * 2] = pack2_bf16(p0, p1);
            pa[j >> 1][(j & 1) * 2 + 1] = pack2_bf16(p2, p3);
        }
        // O += P V: 4 k-steps of 16 keys x 4 channel tiles of 8
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            const int key = 16 * s + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
            for (int p = 0; p < PL; ++p)
#pragma unroll
                for (int np = 0; np < 2; ++np) {
                    uint32_t vb[4];
                    const int q = 2 * np + (lane >> 4);
                    ldmatrix_x4_trans(vbase + p * 4096 + key * 64 + ((q ^ ((key >> 1) & 3)) << 4), vb);
                    mma_bf16(o[p][2 * np], pa[s], vb[0], vb[1]);
                    mma_bf16(o[p][2 * np + 1], pa[s], vb[2], vb[3]);
                }
        }
        __syncthreads();                                              // this stage may be overwritten
    }

    // ---- normalise; stage O^att fp32 [token][32 ch] over the K/V buffers; lse ----
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
    float* stage_o = reinterpret_cast<float*>(smem + gm.off_kv);
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = warp * 16 + g + 8 * r;
        const int t = t0 + row;
        if (t < dm.n_r) {
            const float inv = l_run[r] > 0.f ? 1.f / l_run[r] : 0.f;
#pragma unroll
            for (int p = 0; p < PL; ++p)
#pragma unroll
                for (int n = 0; n < 4; ++n)
                    *reinterpret_cast<float2*>(stage_o + p * (gm.nw * 16 * 32) + row * 32 + 8 * n + 2 * tq) =
                        make_float2(o[p][n][2 * r] * inv, o[p][n][2 * r + 1] * inv);
            if (lse && tq == 0) {
                const int ty = fdiv(t, dm.ws, gm.mul_ws), tx = t - ty * dm.ws;
                lse[((size_t)b * dm.heads + h) * dm.N + (size_t)(y0 + ty) * dm.W + x0 + tx] =
                    (m_run[r] + log2f(l_run[r])) * 0.6931471805599453f;
            }
        }
    }
    __syncthreads();

    // ---- LCE + store: thread = (channel pair, run of 2 tokens along x when ws is even) ----
    {
        const int cp = tid & 15;                                      // channels 2cp, 2cp + 1 of this head
        const int run = (dm.ws & 1) ? 1 : 2;
        const int nruns = (t1 - t0) / run;                            // chunk boundaries are multiples of 16 or n_r
#pragma unroll 1
        for (int p = 0; p < PL; ++p) {                                // one 32-channel plane of the head at a time
            const int hc = (h * PL + p) * 32;                         // first channel of the plane
            float2 wv[25];
            float2 bias2 = make_float2(0.f, 0.f);
            if (dm.lce) {
                const float* wp = lce_w + (size_t)(hc + 2 * cp) * 25;
#pragma unroll
                for (int q = 0; q < 25; ++q) wv[q] = make_float2(__ldg(wp + q), __ldg(wp + 25 + q));
                if (lce_b) bias2 = make_float2(__ldg(lce_b + hc + 2 * cp), __ldg(lce_b + hc + 2 * cp + 1));
            }
            const uint32_t halo = sbase + gm.off_halo + p * (gm.halo_rows * gm.halo_w * 64) + cp * 4;
            const float* stage_p = stage_o + p * (gm.nw * 16 * 32);
            uint32_t* out = reinterpret_cast<uint32_t*>(O) + (img + ch_off) / 4 + p * 16 + cp;
            for (int u = tid >> 4; u < nruns; u += nthreads >> 4) {
                const int t = t0 + u * run;
                const int ty = fdiv(t, dm.ws, gm.mul_ws), tx = t - ty * dm.ws;
                float2 acc[2] = {bias2, bias2};
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
                        const float2 att = *reinterpret_cast<const float2*>(stage_p + (t - t0 + e) * 32 + 2 * cp);
                        const float2 r2 = __fadd2_rn(att, acc[e]);
                        out[((size_t)(y0 + ty) * dm.W + x0 + tx + e) * (dm.C / 2)] = pack2_bf16(r2.x, r2.y);
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------ host side
bool attend_mma_supported(const Dims& d, int dtype) {
    if (dtype != BRA_BF16 || (d.d != 32 && d.d != 64) || d.topk > wm::KCAP) return false;
    const MmaGeom g = mma_geom(d, d.d / 32);
    // the staging tile sits over the K/V buffers; chunk boundaries must not split a token run of the LCE
    if (g.nw * 2048 > g.stages * 8192) return false;
    if (g.chunks > 1 && ((g.nw * 16) % d.ws) != 0) return false;
    if ((long long)d.topk * d.n_r * d.n_r >= (1ll << 32) || d.R > 65535 || d.n_r > 65535) return false;
    return g.smem_bytes <= 200 * 1024 && (long long)d.B * d.R * d.heads * g.chunks < (1ll << 31);
}

cudaError_t launch_attend_mma(const Dims& d, const void* Q, const void* K, const void* V,
                              const int32_t* index, const float* lce_w, const float* lce_b,
                              void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel) {
    const int planes = d.d / 32;
    const MmaGeom g = mma_geom(d, planes);
    auto kernel = planes == 2 ? attend_mma_kernel<2> : attend_mma_kernel<1>;
    static PerDeviceMax smem_set[2];
    cudaError_t e = cudaSuccess;
    if (g.smem_bytes > 48 * 1024)
        e = smem_set[planes - 1].ensure(g.smem_bytes, [&] {
            return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, g.smem_bytes);
        });
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)((long long)d.B * d.R * d.heads * g.chunks);
    e = launch_kernel(kernel, dim3(grid), dim3(g.nw * 32), (size_t)g.smem_bytes, st,
                                  after_own_kernel,
                                  static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(K),
                                  static_cast<const __nv_bfloat16*>(V), index, lce_w, lce_b,
                                  static_cast<__nv_bfloat16*>(O), lse, status, d, g);
    count_launch();
    return e;
}

}  // namespace bra
