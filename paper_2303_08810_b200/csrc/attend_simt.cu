// Token-to-token attention over the routed regions plus LCE on CUDA cores
// (Eq. 6, Eq. 7 with Eq. 1), fp32 arithmetic throughout.  This is the path of
// fp32 problems (an fp32 result to 1e-5 rules out bf16/tf32 tensor-core inputs)
// and the fallback for shapes the tensor-core kernels do not take.
//
// One thread per (query token, head).  The gathered keys K^g / values V^g are
// never formed: the thread walks the k listed regions and reads their tokens'
// rows in place (a warp whose lanes share head and region reads each row once,
// as a broadcast).  Softmax is the one-pass running-max form, rescaled once per
// chunk of 8 keys.
#include "bra_internal.h"

namespace bra {

template <typename T, int D>
__global__ void __launch_bounds__(128)
attend_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                   const int32_t* __restrict__ index, const float* __restrict__ lce_w,
                   const float* __restrict__ lce_b, T* __restrict__ O, float* __restrict__ lse,
                   int32_t* __restrict__ status, Dims dm) {
    // flat thread id -> (b, h, region i, token t in region), t fastest
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

    float q[D], o[D];
    load_row<D>(Q + tok, q);
#pragma unroll
    for (int c = 0; c < D; ++c) { q[c] *= dm.scale; o[c] = 0.f; }
    float m_run = -INFINITY, l_run = 0.f;

    const int hi = dm.heads_i == 1 ? 0 : h;
    const int32_t* row = index + (((size_t)b * dm.heads_i + hi) * dm.R + i) * dm.topk;
    for (int m = 0; m < dm.topk; ++m) {
        const int r = row[m];
        if (r < 0 || r >= dm.R) { record_error(status, BRA_ERR_INDEX, r); continue; }
        const int y0 = (r / dm.S) * dm.hs, x0 = (r % dm.S) * dm.ws;
        for (int j0 = 0; j0 < dm.n_r; j0 += 8) {
            const int nj = dm.n_r - j0 < 8 ? dm.n_r - j0 : 8;
            float s[8];
            float cmax = -INFINITY;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                s[u] = -INFINITY;
                if (u < nj) {
                    const int j = j0 + u;
                    const size_t kt = img + ((size_t)(y0 + j / dm.ws) * dm.W + x0 + j % dm.ws) * dm.C + (size_t)h * D;
                    float kr[D];
                    load_row<D>(K + kt, kr);
                    float acc = 0.f;
#pragma unroll
                    for (int c = 0; c < D; ++c) acc = fmaf(q[c], kr[c], acc);
                    s[u] = acc;
                    cmax = fmaxf(cmax, acc);
                }
            }
            const float m_new = fmaxf(m_run, cmax);
            const float corr = expf(m_run - m_new);      // 0 on the first chunk (m_run = -inf)
            l_run *= corr;
#pragma unroll
            for (int c = 0; c < D; ++c) o[c] *= corr;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (u < nj) {
                    const int j = j0 + u;
                    const size_t kt = img + ((size_t)(y0 + j / dm.ws) * dm.W + x0 + j % dm.ws) * dm.C + (size_t)h * D;
                    const float p = expf(s[u] - m_new);
                    l_run += p;
                    float vr[D];
                    load_row<D>(V + kt, vr);
#pragma unroll
                    for (int c = 0; c < D; ++c) o[c] = fmaf(p, vr[c], o[c]);
                }
            }
            m_run = m_new;
        }
    }
    const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
#pragma unroll
    for (int c = 0; c < D; ++c) o[c] *= inv;
    if (lse) lse[((size_t)b * dm.heads + h) * dm.N + (size_t)y * dm.W + x] = m_run + logf(l_run);

    if (dm.lce) {
        // LCE(V)[y,x,c] = sum_ij w[c,i,j] V[y+i-2, x+j-2, c], zero outside the map
        const float* wh = lce_w + (size_t)h * D * 25;
        for (int ti = 0; ti < 5; ++ti) {
            const int yy = y + ti - 2;
            if (yy < 0 || yy >= dm.H) continue;
            for (int tj = 0; tj < 5; ++tj) {
                const int xx = x + tj - 2;
                if (xx < 0 || xx >= dm.W) continue;
                float vr[D];
                load_row<D>(V + img + ((size_t)yy * dm.W + xx) * dm.C + (size_t)h * D, vr);
#pragma unroll
                for (int c = 0; c < D; ++c) o[c] = fmaf(__ldg(wh + c * 25 + ti * 5 + tj), vr[c], o[c]);
            }
        }
        if (lce_b) {
#pragma unroll
            for (int c = 0; c < D; ++c) o[c] += __ldg(lce_b + h * D + c);
        }
    }
    store_row<D>(O + tok, o);
}

bool attend_simt_supported(const Dims& d) {
    return d.d == 16 || d.d == 32 || d.d == 64 || d.d == 128;
}

template <typename T, int D>
static cudaError_t launch_t(const Dims& d, const void* Q, const void* K, const void* V,
                            const int32_t* index, const float* lce_w, const float* lce_b,
                            void* O, float* lse, int32_t* status, cudaStream_t st) {
    const long long total = (long long)d.B * d.heads * d.R * d.n_r;
    const unsigned blocks = (unsigned)((total + 127) / 128);
    attend_simt_kernel<T, D><<<blocks, 128, 0, st>>>(
        static_cast<const T*>(Q), static_cast<const T*>(K), static_cast<const T*>(V), index,
        lce_w, lce_b, static_cast<T*>(O), lse, status, d);
    count_launch();
    return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_d(const Dims& d, const void* Q, const void* K, const void* V,
                            const int32_t* index, const float* lce_w, const float* lce_b,
                            void* O, float* lse, int32_t* status, cudaStream_t st) {
    switch (d.d) {
        case 16:  return launch_t<T, 16>(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st);
        case 32:  return launch_t<T, 32>(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st);
        case 64:  return launch_t<T, 64>(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st);
        case 128: return launch_t<T, 128>(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_attend_simt(const Dims& d, int dtype, const void* Q, const void* K, const void* V,
                               const int32_t* index, const float* lce_w, const float* lce_b,
                               void* O, float* lse, int32_t* status, cudaStream_t st) {
    if (dtype == BRA_BF16)
        return launch_d<__nv_bfloat16>(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st);
    return launch_d<float>(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st);
}

}  // namespace bra
