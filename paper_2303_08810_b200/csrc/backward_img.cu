// Gradients of the routed attention for a fixed routing index (Eq. 7 with Eq. 1) on small
// feature maps, with one (image, head) of the gathered-from tensors resident in shared memory.
// Same mathematics and the same fixed summation orders as the warp-level kernels that stream
// blocks through shared memory (P recomputed from the saved log-sum-exp; dP = dO V^g^T;
// delta = rowsum(P o dP); dS = P o (dP - delta); dQ = scale dS K^g; dK_j, dV_j summed over the
// query regions that routed to j in the order of the inverse routing index; dV += LCE adjoint),
// but the "gather" is only the row addresses given to ldmatrix:
//   dQ kernel    : CTA = (image, head), K and V slices resident; a warp takes 16 query tokens of a
//                  region, its Q and dO fragments straight from global memory.
//   dK/dV kernel : CTA = (image, head), Q and dO slices resident; a warp takes 16 key tokens of a
//                  region, its K and V fragments from global memory, and walks the queries of the
//                  regions that routed to it; the LCE adjoint reads the resident dO slice.
// No atomics, no CTA-wide barrier after the set-up.
#include "img_common.cuh"

namespace bra {

using namespace ptx;

namespace bimg {
constexpr int MAX_WARPS = 12;
}

struct BwdImgGeom {
    int nw, tpr, units, nblocks;          // nblocks: key blocks of a query tile (dQ kernel)
    uint32_t mul_nr, mul_ws, mul_s, mul_tpr, mul_k;
    int off_a, off_b;                     // the two resident slices
    int off_idx;                          // dQ: routing rows as token ids; dK/dV: inverse offsets [R + 1], then the lists as token ids
    int off_w, off_st, off_stat, smem_bytes;
};

// slice row (img_row_offset) of column lane + 32 e of block blk of a list of region origins (token ids),
// n_r tokens per entry
struct ColGeom {
    bool fixed_t; int mstep; int m_of[2], toff[2];
};
__device__ __forceinline__ ColGeom col_geom(const Dims& dm, const BwdImgGeom& gm, int lane) {
    ColGeom cg;
    cg.fixed_t = (img::KB % dm.n_r) == 0;
    cg.mstep = img::KB / dm.n_r;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int kk = lane + 32 * e;
        cg.m_of[e] = fdiv(kk, dm.n_r, gm.mul_nr);
        const int t = kk - cg.m_of[e] * dm.n_r;
        const int ty = fdiv(t, dm.ws, gm.mul_ws);
        cg.toff[e] = ty * dm.W + (t - ty * dm.ws);
    }
    return cg;
}
__device__ __forceinline__ void col_rows(const ColGeom& cg, const Dims& dm, const BwdImgGeom& gm, const int32_t* list,
                                         int total, int blk, int lane, int trow[2], uint32_t vm[2]) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int kk = blk * img::KB + lane + 32 * e;
        bool valid = kk < total;
        int tr = 0;
        if (valid) {
            int m, off;
            if (cg.fixed_t) {
                m = blk * cg.mstep + cg.m_of[e];
                off = cg.toff[e];
            } else {
                m = fdiv(kk, dm.n_r, gm.mul_nr);
                const int t = kk - m * dm.n_r;
                const int ty = fdiv(t, dm.ws, gm.mul_ws);
                off = ty * dm.W + (t - ty * dm.ws);
            }
            const int base = list[m];
            valid = base >= 0;
            tr = valid ? img_row_offset(base + off) : 0;
        }
        trow[e] = tr;
        vm[e] = __ballot_sync(0xffffffffu, valid);
    }
}

// ------------------------------------------------------------------ dQ and delta
__global__ void __launch_bounds__(bimg::MAX_WARPS * 32, 1)
bwd_dq_img_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                  const __nv_bfloat16* __restrict__ Vg, const int32_t* __restrict__ index,
                  const float* __restrict__ lse, const __nv_bfloat16* __restrict__ dOg,
                  __nv_bfloat16* __restrict__ dQg, float* __restrict__ delta_out,
                  int32_t* __restrict__ inv_off, int32_t* __restrict__ inv_list,
                  int32_t* __restrict__ status, Dims dm, BwdImgGeom gm) {
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = gm.nw * 32;
    const int h = blockIdx.x % dm.heads, b = blockIdx.x / dm.heads;
    const size_t tok_bytes = (size_t)dm.C * 2;
    const size_t row_bytes = (size_t)dm.W * tok_bytes;
    const size_t img_off = (size_t)b * dm.H * row_bytes + (size_t)h * 64;
    const uint8_t* Qb = reinterpret_cast<const uint8_t*>(Qg) + img_off;
    const uint8_t* Gb = reinterpret_cast<const uint8_t*>(dOg) + img_off;
    img_load_slice(sbase + gm.off_a, reinterpret_cast<const uint8_t*>(Kg) + img_off, dm.N, tok_bytes, tid, nthreads);
    img_load_slice(sbase + gm.off_b, reinterpret_cast<const uint8_t*>(Vg) + img_off, dm.N, tok_bytes, tid, nthreads);
    cp_async_commit();
    int32_t* s_idx = reinterpret_cast<int32_t*>(smem + gm.off_idx);
    int32_t* s_raw = s_idx + dm.R * dm.topk;          // the entries as region numbers (-1: bad entry)
    int32_t* s_cnt = s_raw + dm.R * dm.topk;          // [R + 1]
    const int entries = dm.R * dm.topk;
    {
        const int hi = dm.heads_i == 1 ? 0 : h;
        const int32_t* ib = index + ((size_t)b * dm.heads_i + hi) * dm.R * dm.topk;
        for (int e = tid; e < dm.R * dm.topk; e += nthreads) {
            int r = __ldg(ib + e);
            if (r < 0 || r >= dm.R) { record_error(status, BRA_ERR_INDEX, r); r = -1; }
            s_raw[e] = r;
            if (r >= 0) {
                const int qy = fdiv(r, dm.S, gm.mul_s), qx = r - qy * dm.S;
                r = qy * dm.hs * dm.W + qx * dm.ws;
            }
            s_idx[e] = r;
        }
    }
    __syncthreads();
    // Inverse routing index of this (image, routing head) for the dK / dV kernel, while the slices
    // are still in flight: per key region j the query regions whose rows list j, in entry order
    // (query region, then slot) - the fixed order of the dK / dV sums.  Counting by comparison: every
    // thread scans the (few hundred to few thousand) entries in shared memory on its own.
    if (inv_off && (dm.heads_i == dm.heads || h == 0)) {
        const bool by_scan = entries <= 1024;       // few entries: every thread scans them on its own
        // how many entries name region j
        if (by_scan) {
            for (int j = tid; j < dm.R; j += nthreads) {
                int count = 0;
                for (int e = 0; e < entries; ++e) count += s_raw[e] == j;
                s_cnt[j] = count;
            }
        } else {                                    // many: a warp per region, 32 entries at a time, ballots
            for (int j = warp; j < dm.R; j += gm.nw) {
                int count = 0;
                for (int e0 = 0; e0 < entries; e0 += 32) {
                    const int e = e0 + lane;
                    count += __popc(__ballot_sync(0xffffffffu, e < entries && s_raw[e] == j));
                }
                if (lane == 0) s_cnt[j] = count;
            }
        }
        __syncthreads();
        // exclusive prefix over the regions: one warp, a run of regions per lane
        if (warp == 0) {
            const int per = (dm.R + 31) / 32;
            const int j0 = min(lane * per, dm.R), j1 = min(j0 + per, dm.R);
            int sum = 0;
            for (int j = j0; j < j1; ++j) sum += s_cnt[j];
            int incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            int run = incl - sum;
            for (int j = j0; j < j1; ++j) { const int c = s_cnt[j]; s_cnt[j] = run; run += c; }
            if (lane == 31) s_cnt[dm.R] = incl;
        }
        __syncthreads();
        const size_t bh = (size_t)b * dm.heads_i + (dm.heads_i == 1 ? 0 : h);
        int32_t* off = inv_off + bh * (dm.R + 1);
        for (int j = tid; j <= dm.R; j += nthreads) off[j] = s_cnt[j];
        // entry e goes to its region's list at the number of earlier entries that name the same region
        int32_t* outl = inv_list + bh * entries;
        if (by_scan) {
            for (int e = tid; e < entries; e += nthreads) {
                const int r = s_raw[e];
                if (r < 0) continue;
                int rank = 0;
                for (int e2 = 0; e2 < e; ++e2) rank += s_raw[e2] == r;
                outl[s_cnt[r] + rank] = fdiv(e, dm.topk, gm.mul_k);
            }
        } else {
            for (int j = warp; j < dm.R; j += gm.nw) {
                int32_t* lj = outl + s_cnt[j];
                int pos = 0;
                for (int e0 = 0; e0 < entries; e0 += 32) {
                    const int e = e0 + lane;
                    const bool hit = e < entries && s_raw[e] == j;
                    const unsigned m = __ballot_sync(0xffffffffu, hit);
                    if (hit) lj[pos + __popc(m & ((1u << lane) - 1u))] = fdiv(e, dm.topk, gm.mul_k);
                    pos += __popc(m);
                }
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();
    pdl_launch_dependents();          // this CTA's slices are resident: the dK/dV kernel may be set up beside it

    const int g = lane >> 2, tq = lane & 3;
    const float sl2 = dm.scale * 1.4426950408889634f;
    const int total_keys = dm.topk * dm.n_r;
    const uint32_t kbase = sbase + gm.off_a, vbase = sbase + gm.off_b;
    const size_t stat0 = ((size_t)b * dm.heads + h) * dm.N;
    const ColGeom cg = col_geom(dm, gm, lane);
    uint32_t* out = reinterpret_cast<uint32_t*>(dQg) + img_off / 4 + tq;

    for (int u = warp; u < gm.units; u += gm.nw) {
        const int i = fdiv(u, gm.tpr, gm.mul_tpr);
        const int t0 = (u - i * gm.tpr) * 16;
        const int rows = min(16, dm.n_r - t0);
        const int ry = fdiv(i, dm.S, gm.mul_s), rx = i - ry * dm.S;
        const int y0 = ry * dm.hs, x0 = rx * dm.ws;
        const int32_t* irow = s_idx + i * dm.topk;
        uint32_t qa[2][4], ga[2][4];
        img_load_a_global(qa, Qb, y0, x0, t0, rows, dm.ws, gm.mul_ws, row_bytes, tok_bytes, lane);
        img_load_a_global(ga, Gb, y0, x0, t0, rows, dm.ws, gm.mul_ws, row_bytes, tok_bytes, lane);
        bool rvalid[2]; float lse2[2]; size_t spos[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            rvalid[r] = g + 8 * r < rows;
            const int t = rvalid[r] ? t0 + g + 8 * r : 0;
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

        const bool single = gm.nblocks == 1;          // S, P, dP of the only block stay in registers
        const int iters = single ? 1 : 2 * gm.nblocks; // otherwise: one sweep for delta, one for dQ
        for (int it = 0; it < iters; ++it) {
            const int blk = it % gm.nblocks, sweep = it / gm.nblocks;
            int trow[2]; uint32_t vm[2];
            col_rows(cg, dm, gm, irow, total_keys, blk, lane, trow, vm);
            float c[8][4], dp[8][4];
            img_rows_x_gather_t2(c, qa, kbase, dp, ga, vbase, trow, lane);   // S = Q K^T, dP = dO V^T
            // P = exp(S scale - lse); keys that do not count give 0
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t bits = vm[j >> 2] >> (((8 * j) & 31) + 2 * tq);
                const bool fx = bits & 1u, fy = bits & 2u;
                c[j][0] = fx ? ex2_approx(fmaf(c[j][0], sl2, -lse2[0])) : 0.f;
                c[j][1] = fy ? ex2_approx(fmaf(c[j][1], sl2, -lse2[0])) : 0.f;
                c[j][2] = fx ? ex2_approx(fmaf(c[j][2], sl2, -lse2[1])) : 0.f;
                c[j][3] = fy ? ex2_approx(fmaf(c[j][3], sl2, -lse2[1])) : 0.f;
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
                img_frag_x_gather(dq, sa, kbase, trow, lane);   // dQ += dS K
            }
        }
        // dQ = scale * acc; delta kept for the dK/dV kernel
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
}

// ------------------------------------------------------------------ dK, dV
template <int SHAPE>
__global__ void __launch_bounds__(bimg::MAX_WARPS * 32, 1)
bwd_dkv_img_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                   const __nv_bfloat16* __restrict__ Vg, const int32_t* __restrict__ inv_off,
                   const int32_t* __restrict__ inv_list, const float* __restrict__ lse,
                   const float* __restrict__ delta, const __nv_bfloat16* __restrict__ dOg,
                   const float* __restrict__ lce_w, __nv_bfloat16* __restrict__ dKg,
                   __nv_bfloat16* __restrict__ dVg, Dims dm, BwdImgGeom gm) {
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nthreads = gm.nw * 32;
    const int h = blockIdx.x % dm.heads, b = blockIdx.x / dm.heads;
    const size_t tok_bytes = (size_t)dm.C * 2;
    const size_t row_bytes = (size_t)dm.W * tok_bytes;
    const size_t img_off = (size_t)b * dm.H * row_bytes + (size_t)h * 64;
    const uint8_t* Kb = reinterpret_cast<const uint8_t*>(Kg) + img_off;
    const uint8_t* Vb = reinterpret_cast<const uint8_t*>(Vg) + img_off;
    img_load_slice(sbase + gm.off_a, reinterpret_cast<const uint8_t*>(Qg) + img_off, dm.N, tok_bytes, tid, nthreads);
    img_load_slice(sbase + gm.off_b, reinterpret_cast<const uint8_t*>(dOg) + img_off, dm.N, tok_bytes, tid, nthreads);
    cp_async_commit();
    if (dm.lce) img_load_weights(smem + gm.off_w, lce_w + (size_t)h * 32 * 25, true, tid, nthreads);
    // The copies above read inputs of the call and may run beside the dQ kernel (programmatic dependent launch);
    // the inverse routing index and delta are that kernel's: read after the wait, with coherent loads.
    pdl_wait();
    // inverse routing index of this (image, head): offsets, then the query regions as token ids
    int32_t* s_off = reinterpret_cast<int32_t*>(smem + gm.off_idx);
    int32_t* s_list = s_off + dm.R + 1;
    {
        const int hi = dm.heads_i == 1 ? 0 : h;
        const size_t bh = (size_t)b * dm.heads_i + hi;
        for (int e = tid; e <= dm.R; e += nthreads) s_off[e] = __ldcg(inv_off + bh * (dm.R + 1) + e);
        for (int e = tid; e < dm.R * dm.topk; e += nthreads) {
            int r = __ldcg(inv_list + bh * dm.R * dm.topk + e);
            r = min(max(r, 0), dm.R - 1);              // entries past the last list are never read
            const int qy = fdiv(r, dm.S, gm.mul_s), qx = r - qy * dm.S;
            s_list[e] = qy * dm.hs * dm.W + qx * dm.ws;
        }
    }
    cp_async_wait<0>();
    __syncthreads();

    const int g = lane >> 2, tq = lane & 3;
    const float sl2 = dm.scale * 1.4426950408889634f;
    const uint32_t qbase = sbase + gm.off_a, gbase = sbase + gm.off_b;
    const size_t stat0 = ((size_t)b * dm.heads + h) * dm.N;
    const ColGeom cg = col_geom(dm, gm, lane);
    float* stage_v = reinterpret_cast<float*>(smem + gm.off_st) + warp * 16 * 32;   // [16 tokens][32 ch]
    float* st = reinterpret_cast<float*>(smem + gm.off_stat) + warp * 128;          // [64] lse * log2 e, [64] delta
    uint32_t* outk = reinterpret_cast<uint32_t*>(dKg) + img_off / 4 + tq;
    uint32_t* outv = reinterpret_cast<uint32_t*>(dVg) + img_off / 4 + (lane & 15);

    for (int u = warp; u < gm.units; u += gm.nw) {
        const int jr = fdiv(u, gm.tpr, gm.mul_tpr);                 // key region
        const int t0 = (u - jr * gm.tpr) * 16;
        const int rows = min(16, dm.n_r - t0);
        const int ry = fdiv(jr, dm.S, gm.mul_s), rx = jr - ry * dm.S;
        const int y0 = ry * dm.hs, x0 = rx * dm.ws;
        uint32_t ka[2][4], va[2][4];
        img_load_a_global(ka, Kb, y0, x0, t0, rows, dm.ws, gm.mul_ws, row_bytes, tok_bytes, lane);
        img_load_a_global(va, Vb, y0, x0, t0, rows, dm.ws, gm.mul_ws, row_bytes, tok_bytes, lane);
        const int e0 = s_off[jr], e1 = s_off[jr + 1];
        const int32_t* list = s_list + e0;                          // query regions that list jr, fixed order
        const int total_cols = (e1 - e0) * dm.n_r;
        const int nblocks = (total_cols + img::KB - 1) / img::KB;
        float dk[4][4], dv[4][4];
#pragma unroll
        for (int n = 0; n < 4; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) { dk[n][e] = 0.f; dv[n][e] = 0.f; }

        for (int blk = 0; blk < nblocks; ++blk) {
            int trow[2]; uint32_t vm[2];
            col_rows(cg, dm, gm, list, total_cols, blk, lane, trow, vm);
            // statistics of this lane's two columns: fetched now, parked after the first MMAs
            float cl[2], cd[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const bool valid = (vm[e] >> lane) & 1u;
                cl[e] = valid ? __ldg(lse + stat0 + (trow[e] >> 6)) * 1.4426950408889634f : 0.f;   // >> 6: the token
                cd[e] = valid ? __ldcg(delta + stat0 + (trow[e] >> 6)) : 0.f;
            }
            float c[8][4], dp[8][4];
            img_rows_x_gather_t2(c, ka, qbase, dp, va, gbase, trow, lane);   // S^T = K Q^T, dP^T = V dO^T
#pragma unroll
            for (int e = 0; e < 2; ++e) { st[lane + 32 * e] = cl[e]; st[64 + lane + 32 * e] = cd[e]; }
            __syncwarp();
            uint32_t pa[4][4], sa[4][4];                 // P^T and dS^T as A fragments
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int col = 8 * j + 2 * tq;
                const uint32_t bits = vm[j >> 2] >> (((8 * j) & 31) + 2 * tq);
                const bool fx = bits & 1u, fy = bits & 2u;
                const float2 l2 = *reinterpret_cast<const float2*>(st + col);
                const float2 dl = *reinterpret_cast<const float2*>(st + 64 + col);
                const float p0 = fx ? ex2_approx(fmaf(c[j][0], sl2, -l2.x)) : 0.f;
                const float p1 = fy ? ex2_approx(fmaf(c[j][1], sl2, -l2.y)) : 0.f;
                const float p2 = fx ? ex2_approx(fmaf(c[j][2], sl2, -l2.x)) : 0.f;
                const float p3 = fy ? ex2_approx(fmaf(c[j][3], sl2, -l2.y)) : 0.f;
                pa[j >> 1][(j & 1) * 2] = pack2_bf16(p0, p1);
                pa[j >> 1][(j & 1) * 2 + 1] = pack2_bf16(p2, p3);
                sa[j >> 1][(j & 1) * 2] = pack2_bf16(p0 * (dp[j][0] - dl.x), p1 * (dp[j][1] - dl.y));
                sa[j >> 1][(j & 1) * 2 + 1] = pack2_bf16(p2 * (dp[j][2] - dl.x), p3 * (dp[j][3] - dl.y));
            }
            img_frag_x_gather2(dk, sa, qbase, dv, pa, gbase, trow, lane);    // dK += dS^T Q, dV += P^T dO
            __syncwarp();                                        // the statistics may be overwritten
        }

        // dK = scale * acc; dV parked fp32 for the LCE adjoint
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = g + 8 * r;
            if (row < rows) {
                const int t = t0 + row;
                const int ty = fdiv(t, dm.ws, gm.mul_ws), tx = t - ty * dm.ws;
                uint32_t* o = outk + ((size_t)(y0 + ty) * dm.W + x0 + tx) * (dm.C / 2);
#pragma unroll
                for (int n = 0; n < 4; ++n) {
                    o[4 * n] = pack2_bf16(dk[n][2 * r] * dm.scale, dk[n][2 * r + 1] * dm.scale);
                    *reinterpret_cast<float2*>(stage_v + row * 32 + 8 * n + 2 * tq) = make_float2(dv[n][2 * r], dv[n][2 * r + 1]);
                }
            }
        }
        __syncwarp();
        // dV[y, x] += sum_ij w[i, j] dO[y - i + 2, x - j + 2]: the correlation of dO with the flipped filter
        img_lce_store<SHAPE, true>(gbase, dm.lce ? sbase + gm.off_w : 0u, stage_v, outv, t0, rows, y0, x0, dm, gm.mul_ws, lane,
                      make_float2(0.f, 0.f));
        __syncwarp();
    }
}

// ------------------------------------------------------------------ host side
static BwdImgGeom bwd_img_geom(const Dims& d, int nw, bool key_centric) {
    BwdImgGeom g;
    g.nw = nw;
    g.tpr = (d.n_r + 15) / 16;
    g.units = d.R * g.tpr;
    g.nblocks = (d.topk * d.n_r + img::KB - 1) / img::KB;
    g.mul_nr = recip32(d.n_r); g.mul_ws = recip32(d.ws); g.mul_s = recip32(d.S); g.mul_tpr = recip32(g.tpr); g.mul_k = recip32(d.topk);
    int off = 0;
    g.off_a = off;    off += d.N * 64;
    g.off_b = off;    off += d.N * 64;
    g.off_st = off;   off += key_centric ? nw * 2048 : 0;
    g.off_stat = off; off += key_centric ? nw * 512 : 0;
    g.off_w = off;    off += key_centric ? 25 * 16 * 8 : 0;
    g.off_idx = off;  off += (((d.R * d.topk * (key_centric ? 1 : 2) + d.R + 1) * 4 + 15) / 16) * 16;
    g.smem_bytes = off;
    return g;
}

static int bimg_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 1;
    return n;
}

bool backward_img_supported(const Dims& d, int dtype) {
    if (!attend_img_supported(d, dtype)) return false;
    return bwd_img_geom(d, 1, true).smem_bytes <= 200 * 1024;
}

// Warps per CTA: fewest rounds of work, counting a second wave of CTAs and the slower progress of
// a warp on a crowded SM (measured: throughput stops growing near a dozen of these warps per SM).
template <typename Kernel>
static cudaError_t pick_warps(Kernel kernel, const Dims& d, bool key_centric, int* nw_out) {
    const long long grid = (long long)d.B * d.heads;
    const int sms = bimg_sm_count();
    double best = 1e30;
    int best_nw = 0, max_smem = 0;
    for (int nw = 1; nw <= bimg::MAX_WARPS; ++nw)
        if (bwd_img_geom(d, nw, key_centric).smem_bytes <= 200 * 1024) max_smem = bwd_img_geom(d, nw, key_centric).smem_bytes;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    for (int nw = 1; nw <= bimg::MAX_WARPS; ++nw) {
        const BwdImgGeom g = bwd_img_geom(d, nw, key_centric);
        if (g.smem_bytes > 200 * 1024) continue;
        int occ = 0;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, nw * 32, g.smem_bytes)) != cudaSuccess) return e;
        if (occ <= 0) continue;
        const long long slots = (long long)occ * sms;
        const long long per_sm_ctas = grid < slots ? (grid + sms - 1) / sms : occ;
        const double waves = (double)((grid + slots - 1) / slots);
        const double crowd = (double)(per_sm_ctas * nw) / 12.0;
        const double cost = waves * (double)((g.units + nw - 1) / nw) * (crowd > 1.0 ? crowd : 1.0);
        if (cost <= best) { best = cost; best_nw = nw; }
    }
    if (!best_nw) return cudaErrorInvalidConfiguration;
    *nw_out = best_nw;
    return cudaSuccess;
}

cudaError_t launch_backward_img(const Dims& d, const void* Q, const void* K, const void* V,
                                const int32_t* index, const int32_t* inv_off, const int32_t* inv_list,
                                const float* lce_w, const float* lse, const void* dO,
                                void* dQ, void* dK, void* dV, float* delta, int32_t* status, cudaStream_t st) {
    // inv_off / inv_list are written by the dQ kernel here (no separate inverse-index launch)
    const int shape = img_region_shape(d);
    auto dkv_kernel = shape == 44 ? bwd_dkv_img_kernel<44> : shape == 22 ? bwd_dkv_img_kernel<22> : bwd_dkv_img_kernel<0>;
    static thread_local struct { long long grid; int N, ents, dev, nw_q, nw_kv; } memo = {0, 0, 0, -1, 0, 0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorUnknown;
    const long long grid = (long long)d.B * d.heads;
    cudaError_t e;
    if (!(memo.nw_q && memo.grid == grid && memo.N == d.N && memo.ents == d.R * d.topk && memo.dev == dev)) {   // attributes are per device
        int nq = 0, nkv = 0;
        if ((e = pick_warps(bwd_dq_img_kernel, d, false, &nq)) != cudaSuccess) return e;
        if ((e = pick_warps(dkv_kernel, d, true, &nkv)) != cudaSuccess) return e;
        memo.grid = grid; memo.N = d.N; memo.ents = d.R * d.topk; memo.dev = dev; memo.nw_q = nq; memo.nw_kv = nkv;
    }
    const BwdImgGeom a = bwd_img_geom(d, memo.nw_q, false), b = bwd_img_geom(d, memo.nw_kv, true);
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(Q);
    const __nv_bfloat16* k = static_cast<const __nv_bfloat16*>(K);
    const __nv_bfloat16* v = static_cast<const __nv_bfloat16*>(V);
    const __nv_bfloat16* go = static_cast<const __nv_bfloat16*>(dO);
    bwd_dq_img_kernel<<<(unsigned)grid, a.nw * 32, a.smem_bytes, st>>>(q, k, v, index, lse, go, static_cast<__nv_bfloat16*>(dQ),
                                                                    delta, const_cast<int32_t*>(inv_off),
                                                                    const_cast<int32_t*>(inv_list), status, d, a);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    e = launch_kernel(dkv_kernel, dim3((unsigned)grid), dim3(b.nw * 32), (size_t)b.smem_bytes, st, /*after_own_kernel=*/true,
                      q, k, v, inv_off, inv_list, lse, static_cast<const float*>(delta), go, lce_w,
                      static_cast<__nv_bfloat16*>(dK), static_cast<__nv_bfloat16*>(dV), d, b);
    count_launch();
    return e;
}

}  // namespace bra
