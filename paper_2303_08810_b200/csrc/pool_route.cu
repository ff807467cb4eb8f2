// Region-to-region routing (Section 3.2): per-region average of Q and K,
// region affinity A^r = Q^r (K^r)^T (Eq. 4) and row-wise top-k index (Eq. 5).
#include "bra_internal.h"

namespace bra {

// ------------------------------------------------------------------ pooling
// One CTA reduces one region of one image of one tensor.  Thread (x, 16-byte channel
// vector) sums the hs token rows of its column with up to eight independent 16-byte
// loads in flight, parks the partial sums in shared memory, and the CTA then folds the
// ws columns.  Many small CTAs keep a few hundred KB in flight per SM, which is what an
// HBM-bound scan needs.
template <typename T> struct Vec;
template <> struct Vec<float> { static constexpr int n = 4; };
template <> struct Vec<__nv_bfloat16> { static constexpr int n = 8; };

template <typename T>
__global__ void __launch_bounds__(256)
pool_kernel(const T* __restrict__ Q, const T* __restrict__ K,
            float* __restrict__ q_mean, float* __restrict__ k_mean, Dims dm) {
    constexpr int VEC = Vec<T>::n;
    extern __shared__ float part[];   // [ws][C]
    const int r = blockIdx.x, b = blockIdx.y;
    const int ry = r / dm.S, rx = r - ry * dm.S;
    const T* src = blockIdx.z == 0 ? Q : K;
    float* dst = blockIdx.z == 0 ? q_mean : k_mean;
    const int cvecs = dm.C / VEC;
    const int items = dm.ws * cvecs;                       // one token row of the region
    const size_t row_elems = (size_t)dm.W * dm.C;
    const T* reg = src + ((size_t)b * dm.H + (size_t)ry * dm.hs) * row_elems + (size_t)rx * dm.ws * dm.C;

    for (int it = threadIdx.x; it < items; it += blockDim.x) {
        float acc[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
        const T* p = reg + (size_t)it * VEC;               // (x, cvec) in row 0: the region's row is contiguous
        int y = 0;
        for (; y + 8 <= dm.hs; y += 8) {                    // eight loads in flight
            float v[8][VEC];
#pragma unroll
            for (int u = 0; u < 8; ++u) load_row<VEC>(p + (size_t)(y + u) * row_elems, v[u]);
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int i = 0; i < VEC; ++i) acc[i] += v[u][i];
        }
        for (; y < dm.hs; ++y) {
            float v[VEC];
            load_row<VEC>(p + (size_t)y * row_elems, v);
#pragma unroll
            for (int i = 0; i < VEC; ++i) acc[i] += v[i];
        }
#pragma unroll
        for (int i = 0; i < VEC; i += 4)
            *reinterpret_cast<float4*>(&part[it * VEC + i]) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
    }
    __syncthreads();
    pdl_launch_dependents();          // this CTA's loads are done: the next kernel may be set up
    const float inv = 1.0f / (float)dm.n_r;
    for (int c = threadIdx.x; c < dm.C; c += blockDim.x) {
        float s = 0.f;
        for (int x = 0; x < dm.ws; ++x) s += part[x * dm.C + c];
        dst[((size_t)b * dm.R + r) * dm.C + c] = s * inv;
    }
}

// Regions eight token rows high: two threads per (column, 16-byte vector), four rows each, so that a
// region is summed by twice the threads with half the work each (short CTAs turn over faster, which
// is what this latency-bound scan needs).  Row halves are added lower half first.
template <typename T>
__global__ void __launch_bounds__(256)
pool_split_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                  float* __restrict__ q_mean, float* __restrict__ k_mean, Dims dm) {
    constexpr int VEC = Vec<T>::n;
    extern __shared__ float part[];   // [2][ws][C]
    const int r = blockIdx.x, b = blockIdx.y;
    const int ry = r / dm.S, rx = r - ry * dm.S;
    const T* src = blockIdx.z == 0 ? Q : K;
    float* dst = blockIdx.z == 0 ? q_mean : k_mean;
    const int cvecs = dm.C / VEC;
    const int items = dm.ws * cvecs;
    const size_t row_elems = (size_t)dm.W * dm.C;
    const int wsC = dm.ws * dm.C;
    const int it = threadIdx.x % items, yh = threadIdx.x / items;        // blockDim.x == 2 * items
    const T* p = src + ((size_t)b * dm.H + (size_t)ry * dm.hs + 4 * yh) * row_elems + (size_t)rx * dm.ws * dm.C + (size_t)it * VEC;
    float v[4][VEC];
#pragma unroll
    for (int u = 0; u < 4; ++u) load_row<VEC>(p + (size_t)u * row_elems, v[u]);
    float acc[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[i] += v[u][i];
#pragma unroll
    for (int i = 0; i < VEC; i += 4)
        *reinterpret_cast<float4*>(&part[yh * wsC + it * VEC + i]) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
    __syncthreads();
    pdl_launch_dependents();          // this CTA's loads are done: the next kernel may be set up
    const float inv = 1.0f / (float)dm.n_r;
    for (int c = threadIdx.x; c < dm.C; c += blockDim.x) {
        float s = 0.f;
        for (int x = 0; x < dm.ws; ++x) s += part[x * dm.C + c] + part[wsC + x * dm.C + c];
        dst[((size_t)b * dm.R + r) * dm.C + c] = s * inv;
    }
}

// Small square regions (1 x 1, 2 x 2 or 4 x 4 tokens): one CTA per (row of regions, tensor, image); thread = (region of
// that row, 16-byte channel vector) sums all tokens of its region itself - column by column, the rows of a column
// in order, the columns in order: the sums of pool_kernel, bit for bit - so nothing goes through shared memory
// and a CTA moves a whole row of regions.  (One CTA per region is 6 272 CTAs of 64 threads and 2 KB each at the
// stage-3 shape: the launch rate of CTAs, not HBM, sets its time.)
template <typename T, int HS, int WS>
__global__ void __launch_bounds__(512)
pool_rows_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                 float* __restrict__ q_mean, float* __restrict__ k_mean, Dims dm) {
    constexpr int VEC = Vec<T>::n;
    const int ry = blockIdx.x, b = blockIdx.z;
    const T* src = blockIdx.y == 0 ? Q : K;
    float* dst = blockIdx.y == 0 ? q_mean : k_mean;
    const int cvecs = dm.C / VEC;
    const int rx = threadIdx.x / cvecs, cv = threadIdx.x - rx * cvecs;
    if (rx >= dm.S) return;
    const size_t row_elems = (size_t)dm.W * dm.C;
    const T* p = src + ((size_t)b * dm.H + (size_t)ry * HS) * row_elems + (size_t)rx * dm.ws * dm.C + (size_t)cv * VEC;
    // all HS x WS loads of the thread are issued before the first sum
    float v[WS][HS][VEC];
#pragma unroll
    for (int x = 0; x < WS; ++x)
#pragma unroll
        for (int y = 0; y < HS; ++y) load_row<VEC>(p + (size_t)y * row_elems + (size_t)x * dm.C, v[x][y]);
    // the next kernel may be set up from here on: this CTA's loads are out
    pdl_launch_dependents();
    float total[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) total[i] = 0.f;
#pragma unroll
    for (int x = 0; x < WS; ++x) {
        float col[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) col[i] = 0.f;
#pragma unroll
        for (int y = 0; y < HS; ++y)
#pragma unroll
            for (int i = 0; i < VEC; ++i) col[i] += v[x][y][i];
#pragma unroll
        for (int i = 0; i < VEC; ++i) total[i] += col[i];
    }
    const float inv = 1.0f / (float)dm.n_r;
#pragma unroll
    for (int i = 0; i < VEC; ++i) total[i] *= inv;
    store_row<VEC>(dst + ((size_t)b * dm.R + (size_t)ry * dm.S + rx) * dm.C + (size_t)cv * VEC, total);
}

template <typename T>
static cudaError_t launch_pool_rows(const Dims& d, const void* Q, const void* K, float* q_mean, float* k_mean,
                                    cudaStream_t st) {
    const int threads = (d.S * (d.C / Vec<T>::n) + 31) / 32 * 32;
    const dim3 grid(d.S, 2, d.B);
    const T* q = static_cast<const T*>(Q);
    const T* k = static_cast<const T*>(K);
    if (d.hs == 1) pool_rows_kernel<T, 1, 1><<<grid, threads, 0, st>>>(q, k, q_mean, k_mean, d);
    else if (d.hs == 2) pool_rows_kernel<T, 2, 2><<<grid, threads, 0, st>>>(q, k, q_mean, k_mean, d);
    else pool_rows_kernel<T, 4, 4><<<grid, threads, 0, st>>>(q, k, q_mean, k_mean, d);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_pool(const Dims& d, int dtype, const void* Q, const void* K,
                        float* q_mean, float* k_mean, cudaStream_t st) {
    // small regions: a CTA per row of regions
    if ((d.hs == 1 || d.hs == 2 || d.hs == 4) && d.ws == d.hs && d.S * (d.C / (dtype == BRA_BF16 ? 8 : 4)) <= 512 && d.B <= 65535)
        return dtype == BRA_BF16 ? launch_pool_rows<__nv_bfloat16>(d, Q, K, q_mean, k_mean, st)
                                 : launch_pool_rows<float>(d, Q, K, q_mean, k_mean, st);
    const int vec = dtype == BRA_BF16 ? 8 : 4;
    int items = d.ws * (d.C / vec);
    int threads = ((items < 256 ? items : 256) + 31) / 32 * 32;
    size_t smem = sizeof(float) * (size_t)d.ws * d.C;
    dim3 grid(d.R, d.B, 2);
    cudaError_t e;
    if (d.hs == 8 && 2 * items <= 256 && 2 * smem <= 48 * 1024) {
        if (dtype == BRA_BF16)
            pool_split_kernel<__nv_bfloat16><<<grid, 2 * items, 2 * smem, st>>>(
                static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(K), q_mean, k_mean, d);
        else
            pool_split_kernel<float><<<grid, 2 * items, 2 * smem, st>>>(
                static_cast<const float*>(Q), static_cast<const float*>(K), q_mean, k_mean, d);
        count_launch();
        return cudaGetLastError();
    }
    if (dtype == BRA_BF16) {
        if (smem > 48 * 1024 &&
            (e = cudaFuncSetAttribute(pool_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess)
            return e;
        pool_kernel<__nv_bfloat16><<<grid, threads, smem, st>>>(
            static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(K), q_mean, k_mean, d);
    } else {
        if (smem > 48 * 1024 &&
            (e = cudaFuncSetAttribute(pool_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess)
            return e;
        pool_kernel<float><<<grid, threads, smem, st>>>(
            static_cast<const float*>(Q), static_cast<const float*>(K), q_mean, k_mean, d);
    }
    count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ routing
// One CTA per (image, routing head, chunk of 8 affinity rows).  K^r of the head sits in shared memory
// (row stride odd, so a warp reading one row per lane has no bank conflict).
// One warp per affinity row: lane l holds the scores of regions l, l+32, ...;
// the row is sorted by a warp-wide bitonic network on 64-bit keys
//   (order-preserving bits of the fp32 score) << 32 | (0xffffffff - region)
// descending, which yields score-descending, lower-region-first order.
__device__ __forceinline__ uint32_t ordered_bits(float s) {
    s += 0.0f;                                  // -0 -> +0: equal scores tie on the index
    uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int ROWS_PER_CTA = 8;
constexpr int SELECT_MAX_K = 32;            // up to here k rounds of a warp maximum beat the full sort

template <int E>   // E score slots per lane: handles R <= 32 * E
__global__ void __launch_bounds__(256)
route_kernel(const float* q_mean, const float* k_mean, int32_t* __restrict__ index, Dims dm) {
    extern __shared__ float4 ks4[];             // [R][dc + 4] floats: rows 16-byte aligned, conflict-free;
    float* ks = reinterpret_cast<float*>(ks4);  // then this CTA's rows of Q^r, [8][dc]
    pdl_wait();                                  // the means come from the kernel before
    const int b = blockIdx.x / dm.heads_i, h = blockIdx.x % dm.heads_i;
    const int dc = dm.heads_i == 1 ? dm.C : dm.d;   // channels the affinity sums over (a multiple of 4)
    const int c0 = dm.heads_i == 1 ? 0 : h * dm.d;
    const int ld = dc + 4;
    const int dc4 = dc >> 2;
    const float* kb = k_mean + (size_t)b * dm.R * dm.C + c0;
    for (int i = threadIdx.x; i < dm.R * dc4; i += blockDim.x) {
        const int r = i / dc4, c4 = i - r * dc4;
        *reinterpret_cast<float4*>(&ks[r * ld + 4 * c4]) = __ldcg(reinterpret_cast<const float4*>(kb + (size_t)r * dm.C) + c4);
    }
    float* qs = ks + (size_t)dm.R * ld;
    const int row0 = blockIdx.y * ROWS_PER_CTA;
    const float* qb = q_mean + ((size_t)b * dm.R + row0) * dm.C + c0;
    for (int i = threadIdx.x; i < ROWS_PER_CTA * dc4; i += blockDim.x) {
        const int r = i / dc4, c4 = i - r * dc4;
        if (row0 + r < dm.R)
            *reinterpret_cast<float4*>(&qs[r * dc + 4 * c4]) = __ldcg(reinterpret_cast<const float4*>(qb + (size_t)r * dm.C) + c4);
    }
    __syncthreads();
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int i = blockIdx.y * ROWS_PER_CTA + warp; i < dm.R && i < (int)(blockIdx.y + 1) * ROWS_PER_CTA; i += nwarps) {
        // lane l scores candidates l, l + 32, ...: channels in increasing order, one fp32 FMA each
        const float4* qrow = reinterpret_cast<const float4*>(qs + (i - row0) * dc);
        float acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
        for (int c4 = 0; c4 < dc4; ++c4) {
            const float4 q4 = qrow[c4];
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const int j = lane + 32 * e;
                if (j < dm.R) {
                    const float4 k4 = *reinterpret_cast<const float4*>(&ks[j * ld + 4 * c4]);
                    acc[e] = fmaf(q4.x, k4.x, acc[e]);
                    acc[e] = fmaf(q4.y, k4.y, acc[e]);
                    acc[e] = fmaf(q4.z, k4.z, acc[e]);
                    acc[e] = fmaf(q4.w, k4.w, acc[e]);
                }
            }
        }
        unsigned long long key[E];
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int j = lane + 32 * e;
            key[e] = j < dm.R ? ((unsigned long long)ordered_bits(acc[e]) << 32) | (0xffffffffu - (uint32_t)j)
                              : 0ull;
        }
        int32_t* out = index + (((size_t)b * dm.heads_i + h) * dm.R + i) * dm.topk;
        if (dm.topk <= SELECT_MAX_K) {
            // a few winners: one warp-wide maximum per rank (score bits first, then, among the lanes that
            // hold that score, the lower region), the winner's key cleared for the next round
            for (int m = 0; m < dm.topk; ++m) {
                unsigned long long best = key[0];
#pragma unroll
                for (int e = 1; e < E; ++e) best = key[e] > best ? key[e] : best;
                const uint32_t hi = (uint32_t)(best >> 32);
                const uint32_t top_hi = __reduce_max_sync(0xffffffffu, hi);
                const uint32_t lo = hi == top_hi ? (uint32_t)best : 0u;
                const uint32_t top_lo = __reduce_max_sync(0xffffffffu, lo);
                const unsigned long long top = ((unsigned long long)top_hi << 32) | top_lo;
#pragma unroll
                for (int e = 0; e < E; ++e)
                    if (key[e] == top) key[e] = 0ull;        // keys are distinct: they carry the region number
                if (lane == 0) out[m] = (int32_t)(0xffffffffu - top_lo);
            }
            continue;
        }
        // bitonic sort, descending, element id = slot * 32 + lane
#pragma unroll
        for (int k2 = 2; k2 <= 32 * E; k2 <<= 1) {
#pragma unroll
            for (int j = k2 >> 1; j > 0; j >>= 1) {
                if (j >= 32) {
                    const int js = j >> 5;
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        if ((e & js) == 0) {
                            const int id = e * 32 + lane;
                            const bool desc = (id & k2) == 0;
                            unsigned long long a = key[e], c = key[e | js];
                            const bool swap = desc ? (a < c) : (a > c);
                            key[e] = swap ? c : a;
                            key[e | js] = swap ? a : c;
                        }
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const int id = e * 32 + lane;
                        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key[e], j);
                        const bool lower = (id & j) == 0;
                        const bool desc = (id & k2) == 0;
                        const bool keep_max = lower == desc;
                        const unsigned long long mx = key[e] > other ? key[e] : other;
                        const unsigned long long mn = key[e] > other ? other : key[e];
                        key[e] = keep_max ? mx : mn;
                    }
                }
            }
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int rank = e * 32 + lane;
            if (rank < dm.topk) out[rank] = (int32_t)(0xffffffffu - (uint32_t)(key[e] & 0xffffffffull));
        }
    }
}

// Routing of one (image, routing head) by one CTA of 256 threads, for R <= 64 regions and 32 channels per
// routing head - every BiFormer stage with S = 7 or 8.  Three steps with a barrier between them:
//   1. K^r of the head into shared memory; thread (row i = tid & 63, quarter q = tid >> 6) takes its row of
//      Q^r into registers;
//   2. the thread scores candidates j = q, q + 4, ... of its row (Eq. 4: fp32 FMAs over the channels in
//      increasing order, the sums of the other routing kernels), two candidates at a time so that two
//      dependent FMA chains are in flight; a warp reads one K^r row at a time (a broadcast); the
//      order-preserving score bits go to shared memory, [row][65];
//   3. one thread per row picks the top k (Eq. 5) in k passes over two levels (the best of each group of eight
//      candidates in registers, a rescan of the winner's group), higher score first, lower region on ties.
// A warp issues an instruction every five cycles or so in this kind of code, so what counts is the number of
// instructions one warp runs through: against one thread per row for the scores as well (a single 32-FMA
// chain per candidate, 49 candidates) the scores are spread over four times the threads.
constexpr int ROUTE_S_THREADS = 256, ROUTE_S_LD = 36, ROUTE_S_SC = 65;

__global__ void __launch_bounds__(ROUTE_S_THREADS)
route_small_kernel(const float* q_mean, const float* k_mean, int32_t* __restrict__ index, Dims dm) {
    __shared__ __align__(16) float ks[64 * ROUTE_S_LD];
    __shared__ uint32_t sc[64 * ROUTE_S_SC];
    pdl_wait();                                  // the means come from the kernel before
    const int tid = threadIdx.x;
    const int b = blockIdx.x / dm.heads_i, h = blockIdx.x % dm.heads_i;
    const int c0 = dm.heads_i == 1 ? 0 : h * dm.d;
    // ---- 1. K^r slice and this thread's row of Q^r (coherent loads: the pooling kernel may still be draining) ----
    const float* kb = k_mean + (size_t)b * dm.R * dm.C + c0;
    for (int e = tid; e < dm.R * 8; e += ROUTE_S_THREADS) {
        const int r = e >> 3, c4 = e & 7;
        *reinterpret_cast<float4*>(&ks[r * ROUTE_S_LD + 4 * c4]) = __ldcg(reinterpret_cast<const float4*>(kb + (size_t)r * dm.C) + c4);
    }
    const int i = tid & 63, q = tid >> 6;
    float4 qreg[8];
    {
        const float4* qrow = reinterpret_cast<const float4*>(q_mean + ((size_t)b * dm.R + (i < dm.R ? i : 0)) * dm.C + c0);
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) qreg[c4] = __ldcg(qrow + c4);
    }
    for (int e = tid; e < 64 * ROUTE_S_SC; e += ROUTE_S_THREADS) sc[e] = 0u;     // 0: no candidate
    __syncthreads();
    pdl_launch_dependents();
    // ---- 2. scores of candidates q, q + 4, ..., two at a time ----
    for (int j0 = q; j0 < dm.R; j0 += 8) {
        const int j1 = j0 + 4;
        const float4* ka = reinterpret_cast<const float4*>(&ks[(j0 < dm.R ? j0 : 0) * ROUTE_S_LD]);
        const float4* kb4 = reinterpret_cast<const float4*>(&ks[(j1 < dm.R ? j1 : 0) * ROUTE_S_LD]);
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
            const float4 x = ka[c4], y = kb4[c4];
            a0 = fmaf(qreg[c4].x, x.x, a0); a1 = fmaf(qreg[c4].x, y.x, a1);
            a0 = fmaf(qreg[c4].y, x.y, a0); a1 = fmaf(qreg[c4].y, y.y, a1);
            a0 = fmaf(qreg[c4].z, x.z, a0); a1 = fmaf(qreg[c4].z, y.z, a1);
            a0 = fmaf(qreg[c4].w, x.w, a0); a1 = fmaf(qreg[c4].w, y.w, a1);
        }
        // 0 marks "no candidate": real score bits are never 0
        sc[i * ROUTE_S_SC + j0] = ordered_bits(a0);
        if (j1 < dm.R) sc[i * ROUTE_S_SC + j1] = ordered_bits(a1);
    }
    __syncthreads();
    // ---- 3. selection, one thread per row (the other warps are done) ----
    if (tid >= dm.R) return;
    uint32_t* row = sc + tid * ROUTE_S_SC;
    int32_t* out = index + (((size_t)b * dm.heads_i + h) * dm.R + tid) * dm.topk;
    // Two levels: the best of each group of eight candidates stays in registers; a rank costs a maximum over
    // the eight group bests and a rescan of the winner's group only.  Strict comparisons in ascending order:
    // the first of equal scores wins at both levels.
    uint32_t gbest[8];
    int garg[8];
#pragma unroll
    for (int gq = 0; gq < 8; ++gq) {
        gbest[gq] = 0u; garg[gq] = 8 * gq;
#pragma unroll
        for (int tq = 0; tq < 8; ++tq) {
            const uint32_t v = row[8 * gq + tq];
            if (v > gbest[gq]) { gbest[gq] = v; garg[gq] = 8 * gq + tq; }
        }
    }
    for (int m = 0; m < dm.topk; ++m) {
        uint32_t best = gbest[0];
        int arg = garg[0];
#pragma unroll
        for (int gq = 1; gq < 8; ++gq)
            if (gbest[gq] > best) { best = gbest[gq]; arg = garg[gq]; }
        out[m] = arg;
        row[arg] = 0u;
        const int wg = arg >> 3;
        uint32_t nb = 0u;
        int na = 8 * wg;
#pragma unroll
        for (int tq = 0; tq < 8; ++tq) {
            const uint32_t v = row[8 * wg + tq];
            if (v > nb) { nb = v; na = 8 * wg + tq; }
        }
#pragma unroll
        for (int gq = 0; gq < 8; ++gq)
            if (gq == wg) { gbest[gq] = nb; garg[gq] = na; }
    }
}

// Routing with one THREAD per affinity row, for larger k: CTA = (image, routing head, chunk of 64
// rows).  K^r of the head sits in shared memory (read as broadcasts); the thread forms its R scores
// (Eq. 4: fp32 FMAs over the channels in increasing order, the same sums as the warp-per-row
// kernel), parks their order-preserving bits in shared memory and picks the top k by k passes of
// "largest not yet taken, first one on ties" (Eq. 5).  Per row this is a fraction of the
// instructions of k warp-wide reductions.  (Four lanes per row, with a quad reduction per rank,
// measured slower: 28 us against 24 us at 512 image-head pairs, R = 49, k = 16.)
constexpr int ROUTE_T_ROWS = 64;

template <int DC4>   // channels / 4 of a row of Q^r held in registers (8: head dim 32), or 0: any width
__global__ void __launch_bounds__(ROUTE_T_ROWS)
route_rows_kernel(const float* q_mean, const float* k_mean, int32_t* __restrict__ index, Dims dm) {
    extern __shared__ float4 kt4[];             // [R][dc + 4] floats, then [R][64] score bits
    float* ks = reinterpret_cast<float*>(kt4);
    pdl_wait();                                  // the means come from the kernel before
    const int b = blockIdx.x / dm.heads_i, h = blockIdx.x % dm.heads_i;
    const int dc = dm.heads_i == 1 ? dm.C : dm.d;
    const int c0 = dm.heads_i == 1 ? 0 : h * dm.d;
    const int ld = dc + 4;
    const int dc4 = dc >> 2;
    uint32_t* sc = reinterpret_cast<uint32_t*>(ks + (size_t)dm.R * ld) + threadIdx.x;   // this row's scores, stride 64
    const float* kb = k_mean + (size_t)b * dm.R * dm.C + c0;
    // coherent loads: the means come from the pooling kernel this one may overlap
    for (int i = threadIdx.x; i < dm.R * dc4; i += blockDim.x) {
        const int r = i / dc4, c4 = i - r * dc4;
        *reinterpret_cast<float4*>(&ks[r * ld + 4 * c4]) = __ldcg(reinterpret_cast<const float4*>(kb + (size_t)r * dm.C) + c4);
    }
    __syncthreads();
    pdl_launch_dependents();
    const int i = blockIdx.y * ROUTE_T_ROWS + threadIdx.x;
    if (i >= dm.R) return;
    const float4* qrow = reinterpret_cast<const float4*>(q_mean + ((size_t)b * dm.R + i) * dm.C + c0);
    float4 qreg[DC4 > 0 ? DC4 : 1];
#pragma unroll
    for (int c4 = 0; c4 < DC4; ++c4) qreg[c4] = __ldcg(qrow + c4);
    for (int j = 0; j < dm.R; ++j) {
        const float4* krow = reinterpret_cast<const float4*>(&ks[j * ld]);
        float acc = 0.f;
        if (DC4 > 0) {
#pragma unroll
            for (int c4 = 0; c4 < DC4; ++c4) {
                const float4 k4 = krow[c4];
                acc = fmaf(qreg[c4].x, k4.x, acc);
                acc = fmaf(qreg[c4].y, k4.y, acc);
                acc = fmaf(qreg[c4].z, k4.z, acc);
                acc = fmaf(qreg[c4].w, k4.w, acc);
            }
        } else {
            for (int c4 = 0; c4 < dc4; ++c4) {
                const float4 q4 = __ldcg(qrow + c4), k4 = krow[c4];
                acc = fmaf(q4.x, k4.x, acc);
                acc = fmaf(q4.y, k4.y, acc);
                acc = fmaf(q4.z, k4.z, acc);
                acc = fmaf(q4.w, k4.w, acc);
            }
        }
        sc[j * ROUTE_T_ROWS] = ordered_bits(acc);   // never 0 (NaN is canonical after the + 0): 0 marks "taken"
    }
    int32_t* out = index + (((size_t)b * dm.heads_i + h) * dm.R + i) * dm.topk;
    if (dm.R <= 64) {
        // Two levels: the best of each group of eight candidates stays in registers; a rank costs a
        // maximum over the eight group bests and a rescan of the winner's group only.  Strict
        // comparisons in ascending order: the first of equal scores wins at both levels.
        uint32_t gbest[8];
        int garg[8];
#pragma unroll
        for (int gq = 0; gq < 8; ++gq) {
            gbest[gq] = 0u; garg[gq] = 8 * gq;
#pragma unroll
            for (int tq = 0; tq < 8; ++tq) {
                const int j = 8 * gq + tq;
                const uint32_t v = j < dm.R ? sc[j * ROUTE_T_ROWS] : 0u;
                if (v > gbest[gq]) { gbest[gq] = v; garg[gq] = j; }
            }
        }
        for (int m = 0; m < dm.topk; ++m) {
            uint32_t best = gbest[0];
            int arg = garg[0];
#pragma unroll
            for (int gq = 1; gq < 8; ++gq)
                if (gbest[gq] > best) { best = gbest[gq]; arg = garg[gq]; }
            out[m] = arg;
            sc[arg * ROUTE_T_ROWS] = 0u;
            const int wg = arg >> 3;
            uint32_t nb = 0u;
            int na = 8 * wg;
#pragma unroll
            for (int tq = 0; tq < 8; ++tq) {
                const int j = 8 * wg + tq;
                const uint32_t v = j < dm.R ? sc[j * ROUTE_T_ROWS] : 0u;
                if (v > nb) { nb = v; na = j; }
            }
#pragma unroll
            for (int gq = 0; gq < 8; ++gq)
                if (gq == wg) { gbest[gq] = nb; garg[gq] = na; }
        }
        return;
    }
    for (int m = 0; m < dm.topk; ++m) {
        uint32_t best = 0u;
        int arg = 0;
        for (int j = 0; j < dm.R; ++j) {
            const uint32_t v = sc[j * ROUTE_T_ROWS];
            if (v > best) { best = v; arg = j; }    // strict: the first of equal scores wins
        }
        sc[arg * ROUTE_T_ROWS] = 0u;
        out[m] = arg;
    }
}

static size_t route_smem(const Dims& d) {
    const int dc = d.heads_i == 1 ? d.C : d.d;
    return sizeof(float) * ((size_t)d.R * (dc + 4) + (size_t)ROWS_PER_CTA * dc);
}

bool route_supported(const Dims& d) {
    return d.R <= 256 && route_smem(d) <= 200 * 1024 && sizeof(float) * (size_t)d.ws * d.C <= 200 * 1024 &&
           d.B <= 65535;
}

template <int E>
static cudaError_t launch_route_e(const Dims& d, const float* q_mean, const float* k_mean,
                                  int32_t* index, cudaStream_t st) {
    const size_t smem = route_smem(d);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(route_kernel<E>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaError_t e = launch_kernel(route_kernel<E>, dim3(d.B * d.heads_i, (d.R + ROWS_PER_CTA - 1) / ROWS_PER_CTA),
                                  dim3(256), smem, st, /*after_own_kernel=*/true, q_mean, k_mean, index, d);
    count_launch();
    return e;
}

// The same routing with half a warp per affinity row (small R, small k): twice the rows per warp,
// the same instructions per warp.  Lane l of the half scores candidates l, l + 16, ...; the rank
// rounds reduce over the half's 16 lanes (redux with a half-warp mask).
constexpr int HALF_ROWS_PER_CTA = 16;

template <int E2>   // score slots per lane: handles R <= 16 * E2
__global__ void __launch_bounds__(256)
route_half_kernel(const float* q_mean, const float* k_mean, int32_t* __restrict__ index, Dims dm) {
    extern __shared__ float4 kh4[];             // [R][dc + 4] floats, then this CTA's 16 rows of Q^r
    float* ks = reinterpret_cast<float*>(kh4);
    pdl_wait();                                  // the means come from the kernel before
    const int b = blockIdx.x / dm.heads_i, h = blockIdx.x % dm.heads_i;
    const int dc = dm.heads_i == 1 ? dm.C : dm.d;
    const int c0 = dm.heads_i == 1 ? 0 : h * dm.d;
    const int ld = dc + 4;
    const int dc4 = dc >> 2;
    const float* kb = k_mean + (size_t)b * dm.R * dm.C + c0;
    // coherent loads: the means come from the pooling kernel this one may overlap
    for (int i = threadIdx.x; i < dm.R * dc4; i += blockDim.x) {
        const int r = i / dc4, c4 = i - r * dc4;
        *reinterpret_cast<float4*>(&ks[r * ld + 4 * c4]) = __ldcg(reinterpret_cast<const float4*>(kb + (size_t)r * dm.C) + c4);
    }
    float* qs = ks + (size_t)dm.R * ld;
    const int row0 = blockIdx.y * HALF_ROWS_PER_CTA;
    const float* qb = q_mean + ((size_t)b * dm.R + row0) * dm.C + c0;
    for (int i = threadIdx.x; i < HALF_ROWS_PER_CTA * dc4; i += blockDim.x) {
        const int r = i / dc4, c4 = i - r * dc4;
        if (row0 + r < dm.R)
            *reinterpret_cast<float4*>(&qs[r * dc + 4 * c4]) = __ldcg(reinterpret_cast<const float4*>(qb + (size_t)r * dm.C) + c4);
    }
    __syncthreads();
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, l16 = lane & 15, half = lane >> 4;
    const int lrow = (threadIdx.x >> 5) * 2 + half;          // this half-warp's row of the CTA
    const int i = row0 + lrow;
    const bool live = i < dm.R;                               // both halves run the reductions below; a dead one writes nothing
    const unsigned hmask = 0xffffu << (16 * half);
    const float4* qrow = reinterpret_cast<const float4*>(qs + (live ? lrow : 0) * dc);
    float acc[E2];
#pragma unroll
    for (int e = 0; e < E2; ++e) acc[e] = 0.f;
    for (int c4 = 0; c4 < dc4; ++c4) {
        const float4 q4 = qrow[c4];
#pragma unroll
        for (int e = 0; e < E2; ++e) {
            const int j = l16 + 16 * e;
            if (j < dm.R) {
                const float4 k4 = *reinterpret_cast<const float4*>(&ks[j * ld + 4 * c4]);
                acc[e] = fmaf(q4.x, k4.x, acc[e]);
                acc[e] = fmaf(q4.y, k4.y, acc[e]);
                acc[e] = fmaf(q4.z, k4.z, acc[e]);
                acc[e] = fmaf(q4.w, k4.w, acc[e]);
            }
        }
    }
    unsigned long long key[E2];
#pragma unroll
    for (int e = 0; e < E2; ++e) {
        const int j = l16 + 16 * e;
        key[e] = j < dm.R ? ((unsigned long long)ordered_bits(acc[e]) << 32) | (0xffffffffu - (uint32_t)j) : 0ull;
    }
    int32_t* out = index + (((size_t)b * dm.heads_i + h) * dm.R + (live ? i : 0)) * dm.topk;
    for (int m = 0; m < dm.topk; ++m) {
        unsigned long long best = key[0];
#pragma unroll
        for (int e = 1; e < E2; ++e) best = key[e] > best ? key[e] : best;
        const uint32_t hi = (uint32_t)(best >> 32);
        const uint32_t top_hi = __reduce_max_sync(hmask, hi);
        const uint32_t lo = hi == top_hi ? (uint32_t)best : 0u;
        const uint32_t top_lo = __reduce_max_sync(hmask, lo);
        const unsigned long long top = ((unsigned long long)top_hi << 32) | top_lo;
#pragma unroll
        for (int e = 0; e < E2; ++e)
            if (key[e] == top) key[e] = 0ull;            // keys are distinct: they carry the region number
        if (l16 == 0 && live) out[m] = (int32_t)(0xffffffffu - top_lo);
    }
}

static size_t route_half_smem(const Dims& d) {
    const int dc = d.heads_i == 1 ? d.C : d.d;
    return sizeof(float) * ((size_t)d.R * (dc + 4) + (size_t)HALF_ROWS_PER_CTA * dc);
}

template <int E2>
static cudaError_t launch_route_half(const Dims& d, const float* q_mean, const float* k_mean,
                                     int32_t* index, cudaStream_t st) {
    const size_t smem = route_half_smem(d);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(route_half_kernel<E2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaError_t e = launch_kernel(route_half_kernel<E2>, dim3(d.B * d.heads_i, (d.R + HALF_ROWS_PER_CTA - 1) / HALF_ROWS_PER_CTA),
                                  dim3(256), smem, st, /*after_own_kernel=*/true, q_mean, k_mean, index, d);
    count_launch();
    return e;
}

static size_t route_rows_smem(const Dims& d) {
    const int dc = d.heads_i == 1 ? d.C : d.d;
    return sizeof(float) * (size_t)d.R * (dc + 4) + sizeof(uint32_t) * (size_t)d.R * ROUTE_T_ROWS;
}

template <int DC4>
static cudaError_t launch_route_rows(const Dims& d, const float* q_mean, const float* k_mean,
                                     int32_t* index, cudaStream_t st) {
    const size_t smem = route_rows_smem(d);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(route_rows_kernel<DC4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaError_t e = launch_kernel(route_rows_kernel<DC4>, dim3(d.B * d.heads_i, (d.R + ROUTE_T_ROWS - 1) / ROUTE_T_ROWS),
                                  dim3(ROUTE_T_ROWS), smem, st, /*after_own_kernel=*/true, q_mean, k_mean, index, d);
    count_launch();
    return e;
}

cudaError_t launch_route(const Dims& d, const float* q_mean, const float* k_mean,
                         int32_t* index, cudaStream_t st) {
    // up to 64 regions, 32 channels per routing head, more than one winner per row and enough (image, head)
    // pairs for well over one 256-thread CTA per SM: one CTA per pair.  (Measured against the kernels below,
    // pooling + routing: 14.5 against 15.8 us at B = 64, 4 heads, k = 4; 18.6 against 20.6 us at 512 pairs,
    // k = 16; slower with 128 pairs, k = 1 (18.6 against 17.5 us) and with 4 pairs (19.8 against 12.6 us),
    // where one CTA's latency is all there is.)
    if (d.R <= 64 && (d.heads_i == 1 ? d.C : d.d) == 32 && d.topk >= 2 &&
        (long long)d.B * d.heads_i >= 256) {
        cudaError_t e = launch_kernel(route_small_kernel, dim3(d.B * d.heads_i), dim3(ROUTE_S_THREADS), 0, st,
                                      /*after_own_kernel=*/true, q_mean, k_mean, index, d);
        count_launch();
        return e;
    }
    // many winners per row and enough (image, head) pairs to fill the GPU with 64-thread CTAs:
    // one thread per row
    if (d.topk > 8 && (long long)d.B * d.heads_i >= 256 && route_rows_smem(d) <= 100 * 1024) {
        const int dc = d.heads_i == 1 ? d.C : d.d;
        return dc == 32 ? launch_route_rows<8>(d, q_mean, k_mean, index, st)
                        : launch_route_rows<0>(d, q_mean, k_mean, index, st);
    }
    // small R and k: half a warp per row
    if (d.R <= 64 && d.topk <= 8 && route_half_smem(d) <= 100 * 1024)
        return d.R <= 32 ? launch_route_half<2>(d, q_mean, k_mean, index, st)
                         : launch_route_half<4>(d, q_mean, k_mean, index, st);
    if (d.R <= 32) return launch_route_e<1>(d, q_mean, k_mean, index, st);
    if (d.R <= 64) return launch_route_e<2>(d, q_mean, k_mean, index, st);
    if (d.R <= 128) return launch_route_e<4>(d, q_mean, k_mean, index, st);
    return launch_route_e<8>(d, q_mean, k_mean, index, st);
}

// ------------------------------------------------------------------ maps that S does not divide
// The kernels work on maps whose sides are multiples of S; a caller's map of another size is copied into a
// zero-padded one (padding at the bottom and right) and the results are cropped back.  T: uint4 when a
// token's bytes are a multiple of 16, else uint32_t.
template <typename T>
__global__ void __launch_bounds__(256)
pad_copy_kernel(const T* __restrict__ src, T* __restrict__ dst, long long images, int H0, int W0, int H, int W,
                int tvec, bool to_padded) {
    const int Ho = to_padded ? H : H0, Wo = to_padded ? W : W0;        // the map that is written
    const long long total = images * Ho * Wo * tvec;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        const int v = (int)(e % tvec);
        long long t = e / tvec;
        const int x = (int)(t % Wo); t /= Wo;
        const int y = (int)(t % Ho);
        const long long b = t / Ho;
        T val = T();
        if (to_padded) {
            if (y < H0 && x < W0) val = src[((b * H0 + y) * W0 + x) * tvec + v];
        } else {
            val = src[((b * H + y) * W + x) * tvec + v];
        }
        dst[e] = val;
    }
}

cudaError_t launch_pad_copy(const void* src, void* dst, long long images, int H0, int W0, int H, int W,
                            int token_bytes, bool to_padded, cudaStream_t st) {
    const bool wide = token_bytes % 16 == 0 && ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) == 0;
    const int tvec = token_bytes / (wide ? 16 : 4);
    const long long total = images * (to_padded ? (long long)H * W : (long long)H0 * W0) * tvec;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    if (wide)
        pad_copy_kernel<uint4><<<(unsigned)blocks, 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                                                 images, H0, W0, H, W, tvec, to_padded);
    else
        pad_copy_kernel<uint32_t><<<(unsigned)blocks, 256, 0, st>>>(static_cast<const uint32_t*>(src), static_cast<uint32_t*>(dst),
                                                                    images, H0, W0, H, W, tvec, to_padded);
    count_launch();
    return cudaGetLastError();
}

}  // namespace bra
