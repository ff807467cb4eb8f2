// Gradients of O = softmax(scale Q K^g^T) V^g + LCE(V) for a fixed routing
// index (Eq. 7 with Eq. 1; the index of Eq. 5 is a constant), fp32 arithmetic
// on CUDA cores.  Every sum has a fixed order: no atomics on the data path.
//
//   1. inverse index: for each key region, the list (in (query region, slot)
//      order) of query regions that routed to it, as CSR.
//   2. dQ kernel, one thread per (query, head): delta = rowsum(P o dP), then
//      dQ = scale * sum_j P_j (dP_j - delta) K_j; delta is kept for step 3.
//   3. dK/dV kernel, one thread per (key token, head): walks the inverse index,
//      recomputes P from the saved log-sum-exp, accumulates dK, dV, then adds
//      the LCE adjoint dV += sum_ij w[c,i,j] dO[y-i+2, x-j+2, c].
//   4. d_lce_w / d_lce_b: per-CTA partial sums, then a fixed-order final sum.
// Steps 2 and 3 run on the tensor cores instead (backward_mma.cu) for bf16 with head dim 32.
#include "bra_internal.h"
#include "sm100_ptx.cuh"

namespace bra {

// ------------------------------------------------------------ inverse index
// grid: B * heads_i CTAs of 256 threads.  The R * topk entries of the (image, head) are staged
// in shared memory when they fit.  Warp w takes key regions w, w + 8, ...: it sweeps the entries
// 32 at a time and finds its region's hits with a ballot, so the list of a key region comes out
// in entry order (query region, then slot): a fixed order for the dK / dV sums.
__global__ void __launch_bounds__(256)
inverse_index_kernel(const int32_t* __restrict__ index, int32_t* __restrict__ inv_off,
                     int32_t* __restrict__ inv_list, int staged, Dims dm) {
    extern __shared__ int32_t sm[];   // counts[R + 1], then the staged entries
    const int bh = blockIdx.x;
    const int32_t* gidx = index + (size_t)bh * dm.R * dm.topk;
    const int entries = dm.R * dm.topk;
    int32_t* sidx = sm + dm.R + 1;
    if (staged) {
        for (int e = threadIdx.x; e < entries; e += blockDim.x) sidx[e] = gidx[e];
        __syncthreads();
    }
    const int32_t* idx = staged ? sidx : gidx;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int j = warp; j < dm.R; j += nwarps) {
        int count = 0;
        for (int e0 = 0; e0 < entries; e0 += 32) {
            const int e = e0 + lane;
            count += __popc(__ballot_sync(0xffffffffu, e < entries && idx[e] == j));
        }
        if (lane == 0) sm[j] = count;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int r = 0; r < dm.R; ++r) { const int c = sm[r]; sm[r] = run; run += c; }
        sm[dm.R] = run;
    }
    __syncthreads();
    int32_t* off = inv_off + (size_t)bh * (dm.R + 1);
    for (int j = threadIdx.x; j <= dm.R; j += blockDim.x) off[j] = sm[j];
    for (int j = warp; j < dm.R; j += nwarps) {
        int32_t* out = inv_list + (size_t)bh * entries + sm[j];
        int pos = 0;
        for (int e0 = 0; e0 < entries; e0 += 32) {
            const int e = e0 + lane;
            const bool hit = e < entries && idx[e] == j;
            const unsigned m = __ballot_sync(0xffffffffu, hit);
            if (hit) out[pos + __popc(m & ((1u << lane) - 1u))] = e / dm.topk;   // the query region of entry e
            pos += __popc(m);
        }
    }
}

// ------------------------------------------------------------ dQ and delta
template <typename T, int D>
__global__ void __launch_bounds__(128)
bwd_dq_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
              const int32_t* __restrict__ index, const float* __restrict__ lse,
              const T* __restrict__ dO, T* __restrict__ dQ, float* __restrict__ delta,
              int32_t* __restrict__ status, Dims dm) {
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)dm.B * dm.heads * dm.R * dm.n_r;
    if (gid >= total) return;
    const int t = (int)(gid % dm.n_r);
    const int i = (int)((gid / dm.n_r) % dm.R);
    const int h = (int)((gid / ((long long)dm.n_r * dm.R)) % dm.heads);
    const int b = (int)(gid / ((long long)dm.n_r * dm.R * dm.heads));
    const int y = (i / dm.S) * dm.hs + t / dm.ws;
    const int x = (i % dm.S) * dm.ws + t % dm.ws;
    const size_t img = (size_t)b * dm.N * dm.C;
    const size_t tok = img + ((size_t)y * dm.W + x) * dm.C + (size_t)h * D;
    const size_t stat = ((size_t)b * dm.heads + h) * dm.N + (size_t)y * dm.W + x;

    float q[D], go[D], acc[D];
    load_row<D>(Q + tok, q);
    load_row<D>(dO + tok, go);
#pragma unroll
    for (int c = 0; c < D; ++c) { q[c] *= dm.scale; acc[c] = 0.f; }
    const float l = lse[stat];
    const int hi = dm.heads_i == 1 ? 0 : h;
    const int32_t* row = index + (((size_t)b * dm.heads_i + hi) * dm.R + i) * dm.topk;

    float dsum = 0.f;
    for (int pass = 0; pass < 2; ++pass) {
        for (int m = 0; m < dm.topk; ++m) {
            const int r = row[m];
            if (r < 0 || r >= dm.R) { record_error(status, BRA_ERR_INDEX, r); continue; }
            const int y0 = (r / dm.S) * dm.hs, x0 = (r % dm.S) * dm.ws;
            for (int j = 0; j < dm.n_r; ++j) {
                const size_t kt = img + ((size_t)(y0 + j / dm.ws) * dm.W + x0 + j % dm.ws) * dm.C + (size_t)h * D;
                float kr[D], vr[D];
                load_row<D>(K + kt, kr);
                load_row<D>(V + kt, vr);
                float s = 0.f, dp = 0.f;
#pragma unroll
                for (int c = 0; c < D; ++c) { s = fmaf(q[c], kr[c], s); dp = fmaf(go[c], vr[c], dp); }
                const float p = expf(s - l);
                if (pass == 0) {
                    dsum = fmaf(p, dp, dsum);
                } else {
                    const float ds = p * (dp - dsum);
#pragma unroll
                    for (int c = 0; c < D; ++c) acc[c] = fmaf(ds, kr[c], acc[c]);
                }
            }
        }
    }
    delta[stat] = dsum;
#pragma unroll
    for (int c = 0; c < D; ++c) acc[c] *= dm.scale;
    store_row<D>(dQ + tok, acc);
}

// ------------------------------------------------------------ dK, dV
template <typename T, int D>
__global__ void __launch_bounds__(128)
bwd_dkv_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
               const int32_t* __restrict__ inv_off, const int32_t* __restrict__ inv_list,
               const float* __restrict__ lse, const float* __restrict__ delta,
               const T* __restrict__ dO, const float* __restrict__ lce_w,
               T* __restrict__ dK, T* __restrict__ dV, Dims dm) {
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)dm.B * dm.heads * dm.R * dm.n_r;
    if (gid >= total) return;
    const int t = (int)(gid % dm.n_r);
    const int jr = (int)((gid / dm.n_r) % dm.R);          // key region
    const int h = (int)((gid / ((long long)dm.n_r * dm.R)) % dm.heads);
    const int b = (int)(gid / ((long long)dm.n_r * dm.R * dm.heads));
    const int y = (jr / dm.S) * dm.hs + t / dm.ws;
    const int x = (jr % dm.S) * dm.ws + t % dm.ws;
    const size_t img = (size_t)b * dm.N * dm.C;
    const size_t tok = img + ((size_t)y * dm.W + x) * dm.C + (size_t)h * D;

    float kr[D], vr[D], gk[D], gv[D];
    load_row<D>(K + tok, kr);
    load_row<D>(V + tok, vr);
#pragma unroll
    for (int c = 0; c < D; ++c) { kr[c] *= dm.scale; gk[c] = 0.f; gv[c] = 0.f; }

    const int hi = dm.heads_i == 1 ? 0 : h;
    const size_t bh = (size_t)b * dm.heads_i + hi;
    const int32_t* off = inv_off + bh * (dm.R + 1);
    const int32_t* list = inv_list + bh * dm.R * dm.topk;
    const size_t stat0 = ((size_t)b * dm.heads + h) * dm.N;
    for (int e = off[jr]; e < off[jr + 1]; ++e) {
        const int i = list[e];                            // a query region that lists jr
        const int y0 = (i / dm.S) * dm.hs, x0 = (i % dm.S) * dm.ws;
        for (int tq = 0; tq < dm.n_r; ++tq) {
            const int yq = y0 + tq / dm.ws, xq = x0 + tq % dm.ws;
            const size_t qt = img + ((size_t)yq * dm.W + xq) * dm.C + (size_t)h * D;
            float qr[D], go[D];
            load_row<D>(Q + qt, qr);
            load_row<D>(dO + qt, go);
            float s = 0.f, dp = 0.f;
#pragma unroll
            for (int c = 0; c < D; ++c) { s = fmaf(qr[c], kr[c], s); dp = fmaf(go[c], vr[c], dp); }
            const size_t st = stat0 + (size_t)yq * dm.W + xq;
            const float p = expf(s - lse[st]);
            const float ds = p * (dp - delta[st]);
#pragma unroll
            for (int c = 0; c < D; ++c) { gk[c] = fmaf(ds, qr[c], gk[c]); gv[c] = fmaf(p, go[c], gv[c]); }
        }
    }
#pragma unroll
    for (int c = 0; c < D; ++c) gk[c] *= dm.scale;
    if (dm.lce) {
        const float* wh = lce_w + (size_t)h * D * 25;
        for (int ti = 0; ti < 5; ++ti) {
            const int yy = y - ti + 2;
            if (yy < 0 || yy >= dm.H) continue;
            for (int tj = 0; tj < 5; ++tj) {
                const int xx = x - tj + 2;
                if (xx < 0 || xx >= dm.W) continue;
                float go[D];
                load_row<D>(dO + img + ((size_t)yy * dm.W + xx) * dm.C + (size_t)h * D, go);
#pragma unroll
                for (int c = 0; c < D; ++c) gv[c] = fmaf(__ldg(wh + c * 25 + ti * 5 + tj), go[c], gv[c]);
            }
        }
    }
    store_row<D>(dK + tok, gk);
    store_row<D>(dV + tok, gv);
}

// ------------------------------------------------------------ d_lce_w, d_lce_b
// Partial sums: CTA p covers a contiguous range of (image, row) pairs.  Thread (channel pair,
// row slot) keeps the 25 tap sums and the bias sum of its two channels for the rows of its
// slot; the row slots are then added in a fixed order in shared memory.
template <typename T> struct Pair;
template <> struct Pair<float> {
    static __device__ __forceinline__ float2 load(const float* p) { return __ldg(reinterpret_cast<const float2*>(p)); }
};
template <> struct Pair<__nv_bfloat16> {
    static __device__ __forceinline__ float2 load(const __nv_bfloat16* p) {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(p));
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    }
};
// a channel pair as stored (bf16: one 32-bit word; fp32: two floats) and as two floats
template <typename T> struct RawPair;
template <> struct RawPair<float> {
    typedef float2 type;
    static __device__ __forceinline__ float2 load(const float* p) { return __ldg(reinterpret_cast<const float2*>(p)); }
    static __device__ __forceinline__ float2 zero() { return make_float2(0.f, 0.f); }
    static __device__ __forceinline__ float2 unpack(float2 v) { return v; }
};
template <> struct RawPair<__nv_bfloat16> {
    typedef uint32_t type;
    static __device__ __forceinline__ uint32_t load(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const uint32_t*>(p)); }
    static __device__ __forceinline__ uint32_t zero() { return 0u; }
    static __device__ __forceinline__ float2 unpack(uint32_t w) {
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    }
};
constexpr int DW_TI = 5;        // tap rows (blockDim.y)
constexpr int DW_CP = 64;       // channel pairs per pass (blockDim.x at most)

// Partial LCE weight gradient of a strip of rows_per_block image rows:
//   dw[c, ti, tj] += dO[b, y, x, c] * V[b, y + ti - 2, x + tj - 2, c]   (and db[c] += dO)
// Thread = (channel pair, tap row ti): it walks the strip's output rows and, along x, keeps the
// five V values of its tap row under the sliding window in registers (one new load per step),
// so its five sums (tj) take one dO load, one V load and five FMAs per position.  No sums are
// shared between threads: nothing to reduce inside the CTA, and the order of additions is fixed
// (rows ascending, x ascending).  Few registers, many warps: the loads of other warps hide the
// latency of this one's.
template <typename T>
__global__ void __launch_bounds__(DW_CP * DW_TI)
bwd_dw_partial_kernel(const T* __restrict__ V, const T* __restrict__ dO, float* __restrict__ part,
                      int rows_per_block, Dims dm) {
    typedef typename RawPair<T>::type raw_t;
    const long long rows = (long long)dm.B * dm.H;
    const long long r0 = (long long)blockIdx.x * rows_per_block;
    const long long r1 = r0 + rows_per_block < rows ? r0 + rows_per_block : rows;
    const int pairs = dm.C >> 1;
    const int ti = threadIdx.y;
    const size_t tokp = (size_t)dm.C;                      // elements per token
    for (int cp0 = 0; cp0 < pairs; cp0 += blockDim.x) {
        const int cp = cp0 + threadIdx.x;
        if (cp >= pairs) continue;
        float2 acc[5], accb = make_float2(0.f, 0.f);
#pragma unroll
        for (int k = 0; k < 5; ++k) acc[k] = make_float2(0.f, 0.f);
        for (long long r = r0; r < r1; ++r) {
            const int b = (int)(r / dm.H), y = (int)(r - (long long)b * dm.H);
            const int yy = y + ti - 2;
            if (yy < 0 || yy >= dm.H) continue;            // this tap row reads zeros for this output row
            const T* grow = dO + ((size_t)b * dm.N + (size_t)y * dm.W) * tokp + 2 * cp;
            const T* vrow = V + ((size_t)b * dm.N + (size_t)yy * dm.W) * tokp + 2 * cp;
            // window w[k] = V[yy][x + k - 2]; before x = 0: columns -2, -1 are zero, 0 and 1 are loaded
            float2 w0 = make_float2(0.f, 0.f), w1 = w0;
            float2 w2 = RawPair<T>::unpack(RawPair<T>::load(vrow));
            float2 w3 = RawPair<T>::unpack(dm.W > 1 ? RawPair<T>::load(vrow + tokp) : RawPair<T>::zero());
            for (int x0 = 0; x0 < dm.W; x0 += 4) {
                // four positions per trip: their loads go out together
                raw_t nv[4], gr[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int x = x0 + u;
                    nv[u] = x + 2 < dm.W ? RawPair<T>::load(vrow + (size_t)(x + 2) * tokp) : RawPair<T>::zero();
                    gr[u] = x < dm.W ? RawPair<T>::load(grow + (size_t)x * tokp) : RawPair<T>::zero();
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float2 w4 = RawPair<T>::unpack(nv[u]);
                    const float2 g = RawPair<T>::unpack(gr[u]);    // zero beyond the row: adds nothing
                    if (ti == 2) accb = __fadd2_rn(accb, g);
                    acc[0] = __ffma2_rn(g, w0, acc[0]);
                    acc[1] = __ffma2_rn(g, w1, acc[1]);
                    acc[2] = __ffma2_rn(g, w2, acc[2]);
                    acc[3] = __ffma2_rn(g, w3, acc[3]);
                    acc[4] = __ffma2_rn(g, w4, acc[4]);
                    w0 = w1; w1 = w2; w2 = w3; w3 = w4;
                }
            }
        }
        float* out = part + ((size_t)blockIdx.x * dm.C + 2 * cp) * 26;
#pragma unroll
        for (int k = 0; k < 5; ++k) { out[ti * 5 + k] = acc[k].x; out[26 + ti * 5 + k] = acc[k].y; }
        if (ti == 2) { out[25] = accb.x; out[26 + 25] = accb.y; }
    }
}

// a channel pair read from shared memory by 32-bit address, as two floats
template <typename T> struct SmemPair;
template <> struct SmemPair<float> {
    static __device__ __forceinline__ float2 load(uint32_t a) { return ptx::lds_f32x2(a); }
};
template <> struct SmemPair<__nv_bfloat16> {
    static __device__ __forceinline__ float2 load(uint32_t a) {
        const uint32_t w = ptx::lds_u32(a);
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    }
};

// The same sums with the strip's rows of V (rows_per_block + 4) and dO (rows_per_block) copied to
// shared memory first: every byte of the strip is in flight at once, instead of one dependent round
// of global loads per four positions.  Used when the rows fit.
template <typename T>
__global__ void __launch_bounds__(DW_CP * DW_TI)
bwd_dw_partial_staged_kernel(const T* __restrict__ V, const T* __restrict__ dO, float* __restrict__ part,
                             int rows_per_block, Dims dm) {
    typedef typename RawPair<T>::type raw_t;
    extern __shared__ __align__(16) uint8_t dw_smem[];
    const long long rows = (long long)dm.B * dm.H;
    const long long r0 = (long long)blockIdx.x * rows_per_block;
    const long long r1 = r0 + rows_per_block < rows ? r0 + rows_per_block : rows;
    const size_t row_elems = (size_t)dm.W * dm.C;
    const int row_chunks = (int)(row_elems * sizeof(T) / 16);
    T* Vs = reinterpret_cast<T*>(dw_smem);                              // slot s = image row r0 - 2 + s (row space of all images)
    T* Gs = Vs + (size_t)(rows_per_block + 4) * row_elems;
    const int tid = threadIdx.y * blockDim.x + threadIdx.x, nthreads = blockDim.x * blockDim.y;
    const uint32_t vs_addr = ptx::smem_u32(Vs), gs_addr = ptx::smem_u32(Gs);
    for (int s = 0; s < rows_per_block + 4; ++s) {
        const long long rr = r0 - 2 + s;
        if (rr < 0 || rr >= rows) continue;                             // never read: its tap rows are outside the map
        const uint8_t* src = reinterpret_cast<const uint8_t*>(V + (size_t)rr * row_elems);
        for (int c = tid; c < row_chunks; c += nthreads)
            ptx::cp_async_16(vs_addr + (uint32_t)(s * row_chunks + c) * 16, src + (size_t)c * 16, 16);
    }
    for (int s = 0; s < (int)(r1 - r0); ++s) {
        const uint8_t* src = reinterpret_cast<const uint8_t*>(dO + (size_t)(r0 + s) * row_elems);
        for (int c = tid; c < row_chunks; c += nthreads)
            ptx::cp_async_16(gs_addr + (uint32_t)(s * row_chunks + c) * 16, src + (size_t)c * 16, 16);
    }
    ptx::cp_async_commit();
    ptx::cp_async_wait<0>();
    __syncthreads();

    const int pairs = dm.C >> 1;
    const int ti = threadIdx.y;
    const size_t tokp = (size_t)dm.C;
    for (int cp0 = 0; cp0 < pairs; cp0 += blockDim.x) {
        const int cp = cp0 + threadIdx.x;
        if (cp >= pairs) continue;
        float2 acc[5], accb = make_float2(0.f, 0.f);
#pragma unroll
        for (int k = 0; k < 5; ++k) acc[k] = make_float2(0.f, 0.f);
        for (long long r = r0; r < r1; ++r) {
            const int y = (int)(r % dm.H);
            const int yy = y + ti - 2;
            if (yy < 0 || yy >= dm.H) continue;
            // 32-bit shared-memory addresses; the window slides along x, five positions per trip so
            // that the window registers come back to their places without moves
            const uint32_t tb = (uint32_t)(dm.C * sizeof(T));               // bytes per token
            uint32_t pg = gs_addr + (uint32_t)(((r - r0) * row_elems + 2 * cp) * sizeof(T));
            uint32_t pv = vs_addr + (uint32_t)(((r - r0 + ti) * row_elems + 2 * cp) * sizeof(T));
            float2 w0 = make_float2(0.f, 0.f), w1 = w0;
            float2 w2 = SmemPair<T>::load(pv);
            float2 w3 = dm.W > 1 ? SmemPair<T>::load(pv + tb) : make_float2(0.f, 0.f);
            pv += 2 * tb;
            int x = 0;
#define BRA_DW_STEP(WA, WB, WC, WD, WE, G)                 \
            if (ti == 2) accb = __fadd2_rn(accb, G);        \
            acc[0] = __ffma2_rn(G, WA, acc[0]);             \
            acc[1] = __ffma2_rn(G, WB, acc[1]);             \
            acc[2] = __ffma2_rn(G, WC, acc[2]);             \
            acc[3] = __ffma2_rn(G, WD, acc[3]);             \
            acc[4] = __ffma2_rn(G, WE, acc[4]);
            for (; x + 5 <= dm.W - 2; x += 5) {
                float2 g[5], nv[5];
#pragma unroll
                for (int u = 0; u < 5; ++u) { nv[u] = SmemPair<T>::load(pv + u * tb); g[u] = SmemPair<T>::load(pg + u * tb); }
                pv += 5 * tb; pg += 5 * tb;
                BRA_DW_STEP(w0, w1, w2, w3, nv[0], g[0])
                BRA_DW_STEP(w1, w2, w3, nv[0], nv[1], g[1])
                BRA_DW_STEP(w2, w3, nv[0], nv[1], nv[2], g[2])
                BRA_DW_STEP(w3, nv[0], nv[1], nv[2], nv[3], g[3])
                BRA_DW_STEP(nv[0], nv[1], nv[2], nv[3], nv[4], g[4])
                w0 = nv[1]; w1 = nv[2]; w2 = nv[3]; w3 = nv[4];
            }
            for (; x < dm.W; ++x) {
                const float2 w4 = x + 2 < dm.W ? SmemPair<T>::load(pv) : make_float2(0.f, 0.f);
                const float2 g1 = SmemPair<T>::load(pg);
                pv += tb; pg += tb;
                BRA_DW_STEP(w0, w1, w2, w3, w4, g1)
                w0 = w1; w1 = w2; w2 = w3; w3 = w4;
            }
#undef BRA_DW_STEP
        }
        float* out = part + ((size_t)blockIdx.x * dm.C + 2 * cp) * 26;
#pragma unroll
        for (int k = 0; k < 5; ++k) { out[ti * 5 + k] = acc[k].x; out[26 + ti * 5 + k] = acc[k].y; }
        if (ti == 2) { out[25] = accb.x; out[26 + 25] = accb.y; }
    }
}

// Final sum over the partials: 32 outputs per CTA, 32 threads per output each taking every
// 32nd partial in order (four loads in flight); the slice sums are then added in order.
constexpr int DW_SLICES = 32;
__global__ void __launch_bounds__(32 * DW_SLICES)
bwd_dw_final_kernel(const float* __restrict__ part, int blocks,
                    float* __restrict__ d_lce_w, float* __restrict__ d_lce_b, Dims dm) {
    __shared__ float sl[DW_SLICES][32];
    const int o = blockIdx.x * 32 + threadIdx.x;   // (channel, slot)
    const int slice = threadIdx.y;
    const size_t stride = (size_t)dm.C * 26;
    float s = 0.f;
    if (o < dm.C * 26) {
        int p = slice;
        for (; p + 3 * DW_SLICES < blocks; p += 4 * DW_SLICES) {
            const float a0 = part[(size_t)p * stride + o], a1 = part[(size_t)(p + DW_SLICES) * stride + o];
            const float a2 = part[(size_t)(p + 2 * DW_SLICES) * stride + o], a3 = part[(size_t)(p + 3 * DW_SLICES) * stride + o];
            s += a0; s += a1; s += a2; s += a3;
        }
        for (; p < blocks; p += DW_SLICES) s += part[(size_t)p * stride + o];
    }
    sl[slice][threadIdx.x] = s;
    __syncthreads();
    if (slice == 0 && o < dm.C * 26) {
        float t = sl[0][threadIdx.x];
#pragma unroll
        for (int q = 1; q < DW_SLICES; ++q) t += sl[q][threadIdx.x];
        const int c = o / 26, k = o % 26;
        if (k < 25) { if (d_lce_w) d_lce_w[c * 25 + k] = t; }
        else if (d_lce_b) d_lce_b[c] = t;
    }
}

bool backward_supported(const Dims& d) {
    return (d.d == 16 || d.d == 32 || d.d == 64) && d.R <= 1000;
}

// The LCE weight gradient needs only V and dO, the attention gradients need neither of its results: the two
// run side by side (helper stream of bra_internal.h; everything stays on the caller's stream if there is none).
template <typename T, int D>
static cudaError_t launch_bwd_t(const Dims& d, int impl, const void* Q, const void* K, const void* V,
                                const int32_t* index, const float* lce_w, const float* lse,
                                const void* dO, void* dQ, void* dK, void* dV,
                                float* d_lce_w, float* d_lce_b, char* ws, const WsLayout& L,
                                cudaStream_t st) {
    int32_t* status = reinterpret_cast<int32_t*>(ws + L.status);
    float* delta = reinterpret_cast<float*>(ws + L.delta);
    int32_t* inv_off = reinterpret_cast<int32_t*>(ws + L.inv_off);
    int32_t* inv_list = reinterpret_cast<int32_t*>(ws + L.inv_list);
    float* part = reinterpret_cast<float*>(ws + L.dw_part);
    const T* q = static_cast<const T*>(Q); const T* k = static_cast<const T*>(K);
    const T* v = static_cast<const T*>(V); const T* go = static_cast<const T*>(dO);
    cudaError_t e;

    // ---- LCE weight / bias gradient, beside the attention gradients ----
    SideStream* ss = (d.lce || d_lce_b) ? side_stream() : nullptr;
    cudaStream_t dw_st = st;
    if (ss) {
        if (cudaEventRecord(ss->fork, st) != cudaSuccess || cudaStreamWaitEvent(ss->s, ss->fork, 0) != cudaSuccess) ss = nullptr;
        else dw_st = ss->s;
    }
    if (d.lce || d_lce_b) {
        const long long rows = (long long)d.B * d.H;
        const int rpb = (int)((rows + L.dw_blocks - 1) / L.dw_blocks);
        const int nblk = (int)((rows + rpb - 1) / rpb);
        const int cpx = d.C / 2 < DW_CP ? d.C / 2 : DW_CP;
        const size_t dw_smem = (size_t)(2 * rpb + 4) * d.W * d.C * sizeof(T);
        if (dw_smem <= 100 * 1024 && ((size_t)d.W * d.C * sizeof(T)) % 16 == 0) {
            static PerDeviceMax dw_set;
            if (dw_smem > 48 * 1024 &&
                (e = dw_set.ensure((int)dw_smem, [&] {
                     return cudaFuncSetAttribute(bwd_dw_partial_staged_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)dw_smem);
                 })) != cudaSuccess)
                return e;
            bwd_dw_partial_staged_kernel<T><<<nblk, dim3(cpx, DW_TI), dw_smem, dw_st>>>(v, go, part, rpb, d);
        } else {
            bwd_dw_partial_kernel<T><<<nblk, dim3(cpx, DW_TI), 0, dw_st>>>(v, go, part, rpb, d);
        }
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        bwd_dw_final_kernel<<<(d.C * 26 + 31) / 32, dim3(32, DW_SLICES), 0, dw_st>>>(part, nblk, d.lce ? d_lce_w : nullptr, d_lce_b, d);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (ss && cudaEventRecord(ss->join, ss->s) != cudaSuccess) return cudaErrorUnknown;

    // bf16, head dim 32: tensor-core kernels.  Small maps with enough (image, head) pairs to fill the
    // GPU keep a whole slice resident; the rest stream blocks through shared memory.
    const bool img_ok = sizeof(T) == 2 && backward_img_supported(d, BRA_BF16);
    const bool use_img = img_ok && (impl == BRA_IMPL_IMG ||
                                    (impl == BRA_IMPL_AUTO && (long long)d.B * d.heads >= 64));
    if (!use_img) {
        const int thr = 256;
        const size_t idx_bytes = sizeof(int32_t) * (size_t)d.R * d.topk;
        const int staged = idx_bytes <= 40 * 1024;
        inverse_index_kernel<<<d.B * d.heads_i, thr, sizeof(int32_t) * (d.R + 1) + (staged ? idx_bytes : 0), st>>>(
            index, inv_off, inv_list, staged, d);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (use_img) {
        // the dQ kernel of this family also writes the inverse routing index
        if ((e = launch_backward_img(d, Q, K, V, index, inv_off, inv_list, lce_w, lse, dO, dQ, dK, dV,
                                     delta, status, st)) != cudaSuccess) return e;
    } else if (sizeof(T) == 2 && impl != BRA_IMPL_SIMT && backward_mma_supported(d, BRA_BF16)) {
        // head dim 32, bf16: the two tensor-core kernels (dQ + delta, then dK / dV)
        if ((e = launch_backward_mma(d, Q, K, V, index, inv_off, inv_list, lce_w, lse, dO, dQ, dK, dV,
                                     delta, status, st)) != cudaSuccess) return e;
    } else {
        const long long total = (long long)d.B * d.heads * d.R * d.n_r;
        const unsigned blocks = (unsigned)((total + 127) / 128);
        bwd_dq_kernel<T, D><<<blocks, 128, 0, st>>>(q, k, v, index, lse, go, static_cast<T*>(dQ), delta, status, d);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;

        bwd_dkv_kernel<T, D><<<blocks, 128, 0, st>>>(q, k, v, inv_off, inv_list, lse, delta, go, lce_w,
                                                     static_cast<T*>(dK), static_cast<T*>(dV), d);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }

    if (ss && cudaStreamWaitEvent(st, ss->join, 0) != cudaSuccess) return cudaErrorUnknown;
    return cudaSuccess;
}

template <typename T>
static cudaError_t launch_bwd_d(const Dims& d, int impl, const void* Q, const void* K, const void* V,
                                const int32_t* index, const float* lce_w, const float* lse,
                                const void* dO, void* dQ, void* dK, void* dV,
                                float* d_lce_w, float* d_lce_b, char* ws, const WsLayout& L,
                                cudaStream_t st) {
    switch (d.d) {
        case 16: return launch_bwd_t<T, 16>(d, impl, Q, K, V, index, lce_w, lse, dO, dQ, dK, dV, d_lce_w, d_lce_b, ws, L, st);
        case 32: return launch_bwd_t<T, 32>(d, impl, Q, K, V, index, lce_w, lse, dO, dQ, dK, dV, d_lce_w, d_lce_b, ws, L, st);
        case 64: return launch_bwd_t<T, 64>(d, impl, Q, K, V, index, lce_w, lse, dO, dQ, dK, dV, d_lce_w, d_lce_b, ws, L, st);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_backward(const Dims& d, int dtype, int impl, const void* Q, const void* K, const void* V,
                            const int32_t* index, const float* lce_w, const float* lse,
                            const void* dO, void* dQ, void* dK, void* dV,
                            float* d_lce_w, float* d_lce_b,
                            char* ws, const WsLayout& L, cudaStream_t st) {
    if (dtype == BRA_BF16)
        return launch_bwd_d<__nv_bfloat16>(d, impl, Q, K, V, index, lce_w, lse, dO, dQ, dK, dV, d_lce_w, d_lce_b, ws, L, st);
    return launch_bwd_d<float>(d, impl, Q, K, V, index, lce_w, lse, dO, dQ, dK, dV, d_lce_w, d_lce_b, ws, L, st);
}

}  // namespace bra
