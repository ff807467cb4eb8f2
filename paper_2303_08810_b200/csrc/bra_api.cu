// Host side of the C boundary: argument checks, scratch layout, kernel choice.
#include "bra_internal.h"

#include <math.h>

namespace bra {

static thread_local int g_launches = 0;
void count_launch(int n) { g_launches += n; }

static size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

WsLayout ws_layout(const Dims& d) {
    WsLayout L;
    size_t off = 0;
    L.status = off;   off += 256;
    L.q_mean = off;   off += align256(sizeof(float) * (size_t)d.B * d.R * d.C);
    L.k_mean = off;   off += align256(sizeof(float) * (size_t)d.B * d.R * d.C);
    L.index = off;    off += align256(sizeof(int32_t) * (size_t)d.B * d.heads_i * d.R * d.topk);
    L.delta = off;    off += align256(sizeof(float) * (size_t)d.B * d.heads * d.N);
    L.inv_off = off;  off += align256(sizeof(int32_t) * (size_t)d.B * d.heads_i * (d.R + 1));
    L.inv_list = off; off += align256(sizeof(int32_t) * (size_t)d.B * d.heads_i * d.R * d.topk);
    // one partial per (image, region row), capped so the scratch stays small
    int blocks = d.B * d.S;
    while (blocks > 1024 && blocks % 2 == 0) blocks /= 2;
    L.dw_blocks = blocks;
    L.dw_part = off;  off += align256(sizeof(float) * (size_t)blocks * d.C * 26);
    L.pad = L.pad_lse = off;
    L.pad_tensor = 0;
    if (d.H != d.H0 || d.W != d.W0) {
        L.pad_tensor = align256((size_t)d.B * d.N * d.C * d.esize);
        L.pad = off;      off += 7 * L.pad_tensor;
        L.pad_lse = off;  off += align256(sizeof(float) * (size_t)d.B * d.heads * d.N);
    }
    L.total = off;
    return L;
}

// Validate the problem statement; fill the derived dimensions.
static bra_status make_dims(const bra_problem* p, Dims* out) {
    if (!p) return BRA_ERR_NULL;
    if (p->B <= 0 || p->H <= 0 || p->W <= 0 || p->C <= 0 || p->heads <= 0 || p->S <= 0)
        return BRA_ERR_SHAPE;
    if (p->C % p->heads) return BRA_ERR_SHAPE;
    // S need not divide H, W: the map is zero-padded at the bottom and right to the next multiples of S
    const int Hp = (p->H + p->S - 1) / p->S * p->S, Wp = (p->W + p->S - 1) / p->S * p->S;
    if ((int64_t)p->B * Hp * Wp * p->C >= ((int64_t)1 << 40)) return BRA_ERR_SHAPE;
    if (p->topk < 1 || (int64_t)p->topk > (int64_t)p->S * p->S) return BRA_ERR_TOPK;
    if (p->dtype != BRA_F32 && p->dtype != BRA_BF16) return BRA_ERR_DTYPE;
    if (p->lce_ksize != 0 && p->lce_ksize != 5) return BRA_ERR_UNSUPPORTED;
    if (p->impl < BRA_IMPL_AUTO || p->impl > BRA_IMPL_TC_FUSED) return BRA_ERR_UNSUPPORTED;
    if (p->inject != BRA_INJECT_NONE && p->inject != BRA_INJECT_LOSE_POOLED_UNIT) return BRA_ERR_UNSUPPORTED;
    Dims d;
    d.B = p->B; d.H = Hp; d.W = Wp; d.C = p->C; d.heads = p->heads; d.S = p->S; d.topk = p->topk;
    d.H0 = p->H; d.W0 = p->W;
    d.esize = p->dtype == BRA_BF16 ? 2 : 4;
    d.d = p->C / p->heads;
    d.R = p->S * p->S;
    d.hs = Hp / p->S; d.ws = Wp / p->S;
    d.n_r = d.hs * d.ws;
    d.N = Hp * Wp;
    d.heads_i = p->shared_routing ? 1 : p->heads;
    d.lce = p->lce_ksize == 5;
    d.scale = p->scale > 0.f ? p->scale : 1.0f / sqrtf((float)d.d);
    // 16-byte vector access to a head's channel slice
    const int vec = p->dtype == BRA_BF16 ? 8 : 4;
    if (d.d % vec) return BRA_ERR_UNSUPPORTED;
    *out = d;
    return BRA_OK;
}

// For translation units that add entry points of their own.
bra_status check_problem(const bra_problem* p, Dims* out) { return make_dims(p, out); }
void reset_launch_count() { g_launches = 0; }

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

static bra_status check_ws(const Dims& d, const void* ws, size_t ws_bytes, WsLayout* L) {
    if (!ws) return BRA_ERR_NULL;
    if (!aligned(ws, 256)) return BRA_ERR_ALIGN;
    *L = ws_layout(d);
    if (ws_bytes < L->total) return BRA_ERR_WORKSPACE;
    return BRA_OK;
}

SideStream* side_stream() {
    static const bool off = getenv("BRA_NO_SIDE_STREAM") != nullptr;
    if (off) return nullptr;
    static thread_local SideStream made[64];
    static thread_local int state[64] = {};            // 0: not tried, 1: ready, 2: failed
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (state[dev] == 0) {
        SideStream& m = made[dev];
        const bool ok = cudaStreamCreateWithFlags(&m.s, cudaStreamNonBlocking) == cudaSuccess &&
                        cudaEventCreateWithFlags(&m.fork, cudaEventDisableTiming) == cudaSuccess &&
                        cudaEventCreateWithFlags(&m.join, cudaEventDisableTiming) == cudaSuccess;
        state[dev] = ok ? 1 : 2;
    }
    return state[dev] == 1 ? &made[dev] : nullptr;
}

static bool padded(const Dims& d) { return d.H != d.H0 || d.W != d.W0; }

// The zero-padded copy of a caller's map in slot `slot` of the scratch buffer (or the map itself if S divides it).
static const void* pad_in(const Dims& d, const WsLayout& L, char* w, int slot, const void* src, cudaStream_t st, bool* ok) {
    if (!padded(d)) return src;
    void* dst = w + L.pad + slot * L.pad_tensor;
    if (launch_pad_copy(src, dst, d.B, d.H0, d.W0, d.H, d.W, d.C * d.esize, true, st) != cudaSuccess) *ok = false;
    return dst;
}
static void* pad_out(const Dims& d, const WsLayout& L, char* w, int slot, void* dst) {
    return padded(d) ? static_cast<void*>(w + L.pad + slot * L.pad_tensor) : dst;
}
static void crop_out(const Dims& d, const WsLayout& L, char* w, int slot, void* dst, cudaStream_t st, bool* ok) {
    if (!padded(d) || !dst) return;
    if (launch_pad_copy(w + L.pad + slot * L.pad_tensor, dst, d.B, d.H0, d.W0, d.H, d.W, d.C * d.esize, false, st) != cudaSuccess)
        *ok = false;
}

enum Path { PATH_NONE, PATH_SIMT, PATH_MMA, PATH_TC, PATH_TC_WIDE, PATH_IMG };

static Path choose_attend(const Dims& d, int dtype, int impl) {
    switch (impl) {
        case BRA_IMPL_SIMT: return attend_simt_supported(d) ? PATH_SIMT : PATH_NONE;
        case BRA_IMPL_MMA:  return attend_mma_supported(d, dtype) ? PATH_MMA : PATH_NONE;
        case BRA_IMPL_TC_FUSED: return attend_tc_supported(d, dtype) ? PATH_TC : PATH_NONE;
        case BRA_IMPL_TC:   return attend_tc_supported(d, dtype) ? PATH_TC
                                 : attend_tc_wide_supported(d, dtype) ? PATH_TC_WIDE : PATH_NONE;
        case BRA_IMPL_IMG:  return attend_img_supported(d, dtype) ? PATH_IMG : PATH_NONE;
        default: break;
    }
    if (attend_tc_supported(d, dtype)) return PATH_TC;
    if (attend_tc_wide_supported(d, dtype)) return PATH_TC_WIDE;
    // one CTA per (image, head): worth it once those fill a good part of the GPU
    if (attend_img_supported(d, dtype) && (long long)d.B * d.heads >= 64) return PATH_IMG;
    if (attend_mma_supported(d, dtype)) return PATH_MMA;
    if (attend_simt_supported(d)) return PATH_SIMT;
    return PATH_NONE;
}

static bra_status run_route(const Dims& d, int dtype, const void* Q, const void* K,
                            float* q_mean, float* k_mean, int32_t* index, cudaStream_t st) {
    if (launch_pool(d, dtype, Q, K, q_mean, k_mean, st) != cudaSuccess) return BRA_ERR_CUDA;
    if (launch_route(d, q_mean, k_mean, index, st) != cudaSuccess) return BRA_ERR_CUDA;
    return BRA_OK;
}

static bra_status run_attend(Path path, const Dims& d, int dtype, const void* Q, const void* K,
                             const void* V, const int32_t* index, const float* lce_w,
                             const float* lce_b, void* O, float* lse, int32_t* status,
                             cudaStream_t st, bool after_own_kernel) {
    cudaError_t e = cudaErrorInvalidValue;
    switch (path) {
        case PATH_SIMT: e = launch_attend_simt(d, dtype, Q, K, V, index, lce_w, lce_b, O, lse, status, st); break;
        case PATH_MMA:  e = launch_attend_mma(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st, after_own_kernel); break;
        case PATH_TC:   e = launch_attend_tc(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st, after_own_kernel); break;
        case PATH_TC_WIDE: e = launch_attend_tc_wide(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st, after_own_kernel); break;
        case PATH_IMG:  e = launch_attend_img(d, Q, K, V, index, lce_w, lce_b, O, lse, status, st, after_own_kernel); break;
        default: return BRA_ERR_UNSUPPORTED;
    }
    return e == cudaSuccess ? BRA_OK : BRA_ERR_CUDA;
}

}  // namespace bra

using namespace bra;

extern "C" {

size_t bra_workspace_bytes(const bra_problem* p) {
    Dims d;
    if (make_dims(p, &d) != BRA_OK) return 0;
    return ws_layout(d).total;
}

bra_status bra_route(const bra_problem* p, const void* Q, const void* K,
                     float* q_mean, float* k_mean, int32_t* index,
                     void* ws, size_t ws_bytes, void* stream) {
    g_launches = 0;
    Dims d;
    bra_status s = make_dims(p, &d);
    if (s != BRA_OK) return s;
    if (!Q || !K || !index) return BRA_ERR_NULL;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(index, 16) ||
        !aligned(q_mean, 16) || !aligned(k_mean, 16)) return BRA_ERR_ALIGN;
    WsLayout L;
    if ((s = check_ws(d, ws, ws_bytes, &L)) != BRA_OK) return s;
    if (!route_supported(d)) return BRA_ERR_UNSUPPORTED;
    char* w = static_cast<char*>(ws);
    float* qm = q_mean ? q_mean : reinterpret_cast<float*>(w + L.q_mean);
    float* km = k_mean ? k_mean : reinterpret_cast<float*>(w + L.k_mean);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    bool ok = true;
    Q = pad_in(d, L, w, 0, Q, st, &ok);
    K = pad_in(d, L, w, 1, K, st, &ok);
    if (!ok) return BRA_ERR_CUDA;
    return run_route(d, p->dtype, Q, K, qm, km, index, st);
}

bra_status bra_attend(const bra_problem* p, const void* Q, const void* K, const void* V,
                      const int32_t* index, const float* lce_w, const float* lce_b,
                      void* O, float* lse, void* ws, size_t ws_bytes, void* stream) {
    g_launches = 0;
    Dims d;
    bra_status s = make_dims(p, &d);
    if (s != BRA_OK) return s;
    if (!Q || !K || !V || !index || !O) return BRA_ERR_NULL;
    if (d.lce && !lce_w) return BRA_ERR_NULL;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) ||
        !aligned(index, 4) || !aligned(lce_w, 4) || !aligned(lce_b, 4) || !aligned(lse, 4))
        return BRA_ERR_ALIGN;
    WsLayout L;
    if ((s = check_ws(d, ws, ws_bytes, &L)) != BRA_OK) return s;
    Path path = choose_attend(d, p->dtype, p->impl);
    if (path == PATH_NONE) return BRA_ERR_UNSUPPORTED;
    char* w = static_cast<char*>(ws);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    bool ok = true;
    Q = pad_in(d, L, w, 0, Q, st, &ok);
    K = pad_in(d, L, w, 1, K, st, &ok);
    V = pad_in(d, L, w, 2, V, st, &ok);
    if (!ok) return BRA_ERR_CUDA;
    float* lse_k = (lse && padded(d)) ? reinterpret_cast<float*>(w + L.pad_lse) : lse;
    s = run_attend(path, d, p->dtype, Q, K, V, index, lce_w, lce_b, pad_out(d, L, w, 3, O), lse_k,
                   reinterpret_cast<int32_t*>(w + L.status), st, false);
    if (s != BRA_OK) return s;
    crop_out(d, L, w, 3, O, st, &ok);
    if (lse && padded(d) &&
        launch_pad_copy(lse_k, lse, (long long)d.B * d.heads, d.H0, d.W0, d.H, d.W, 4, false, st) != cudaSuccess) ok = false;
    return ok ? BRA_OK : BRA_ERR_CUDA;
}

bra_status bra_forward(const bra_problem* p, const void* Q, const void* K, const void* V,
                       const float* lce_w, const float* lce_b, void* O,
                       int32_t* index, float* lse, void* ws, size_t ws_bytes, void* stream) {
    g_launches = 0;
    Dims d;
    bra_status s = make_dims(p, &d);
    if (s != BRA_OK) return s;
    if (!Q || !K || !V || !O) return BRA_ERR_NULL;
    if (d.lce && !lce_w) return BRA_ERR_NULL;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) ||
        !aligned(index, 16) || !aligned(lce_w, 4) || !aligned(lce_b, 4) || !aligned(lse, 4))
        return BRA_ERR_ALIGN;
    WsLayout L;
    if ((s = check_ws(d, ws, ws_bytes, &L)) != BRA_OK) return s;
    if (!route_supported(d)) return BRA_ERR_UNSUPPORTED;
    Path path = choose_attend(d, p->dtype, p->impl);
    if (path == PATH_NONE) return BRA_ERR_UNSUPPORTED;
    char* w = static_cast<char*>(ws);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* idx = index ? index : reinterpret_cast<int32_t*>(w + L.index);
    int32_t* status = reinterpret_cast<int32_t*>(w + L.status);
    float* qm = reinterpret_cast<float*>(w + L.q_mean);
    float* km = reinterpret_cast<float*>(w + L.k_mean);
    bool ok = true;
    Q = pad_in(d, L, w, 0, Q, st, &ok);
    K = pad_in(d, L, w, 1, K, st, &ok);
    V = pad_in(d, L, w, 2, V, st, &ok);
    if (!ok) return BRA_ERR_CUDA;
    void* O_user = O;
    float* lse_user = lse;
    O = pad_out(d, L, w, 3, O);
    if (lse && padded(d)) lse = reinterpret_cast<float*>(w + L.pad_lse);
    auto finish = [&](bra_status rs) -> bra_status {
        if (rs != BRA_OK) return rs;
        crop_out(d, L, w, 3, O_user, st, &ok);
        if (lse_user && padded(d) &&
            launch_pad_copy(lse, lse_user, (long long)d.B * d.heads, d.H0, d.W0, d.H, d.W, 4, false, st) != cudaSuccess) ok = false;
        return ok ? BRA_OK : BRA_ERR_CUDA;
    };
    // pooling, routing and attention in one launch
    static const bool one_launch = getenv("BRA_ONE_LAUNCH") != nullptr;     // tuning aid: also under BRA_IMPL_AUTO
    if (p->impl == BRA_IMPL_TC_FUSED && !forward_tc_supported(d, p->dtype)) return BRA_ERR_UNSUPPORTED;
    if (p->impl == BRA_IMPL_TC_FUSED ||
        (one_launch && p->impl == BRA_IMPL_AUTO && path == PATH_TC && forward_tc_supported(d, p->dtype))) {
        const cudaError_t e = launch_forward_tc(d, Q, K, V, lce_w, lce_b, O, idx, lse, qm, km, status, p->inject, st);
        return finish(e == cudaSuccess ? BRA_OK : BRA_ERR_CUDA);
    }
    s = run_route(d, p->dtype, Q, K, qm, km, idx, st);
    if (s != BRA_OK) return s;
    return finish(run_attend(path, d, p->dtype, Q, K, V, idx, lce_w, lce_b, O, lse, status, st, true));
}

bra_status bra_backward(const bra_problem* p, const void* Q, const void* K, const void* V,
                        const int32_t* index, const float* lce_w, const float* lse,
                        const void* dO, void* dQ, void* dK, void* dV,
                        float* d_lce_w, float* d_lce_b,
                        void* ws, size_t ws_bytes, void* stream) {
    g_launches = 0;
    Dims d;
    bra_status s = make_dims(p, &d);
    if (s != BRA_OK) return s;
    if (!Q || !K || !V || !index || !lse || !dO || !dQ || !dK || !dV) return BRA_ERR_NULL;
    if (d.lce && (!lce_w || !d_lce_w)) return BRA_ERR_NULL;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(dO, 16) ||
        !aligned(dQ, 16) || !aligned(dK, 16) || !aligned(dV, 16) || !aligned(index, 4) ||
        !aligned(lse, 4) || !aligned(lce_w, 4) || !aligned(d_lce_w, 4) || !aligned(d_lce_b, 4))
        return BRA_ERR_ALIGN;
    WsLayout L;
    if ((s = check_ws(d, ws, ws_bytes, &L)) != BRA_OK) return s;
    if (!backward_supported(d)) return BRA_ERR_UNSUPPORTED;
    char* w = static_cast<char*>(ws);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    bool ok = true;
    Q = pad_in(d, L, w, 0, Q, st, &ok);
    K = pad_in(d, L, w, 1, K, st, &ok);
    V = pad_in(d, L, w, 2, V, st, &ok);
    dO = pad_in(d, L, w, 3, dO, st, &ok);          // zero in the padding: padded queries contribute nothing
    if (padded(d)) {                               // lse of the padded queries: 0 (their scores are 0, their P finite)
        float* lp = reinterpret_cast<float*>(w + L.pad_lse);
        if (launch_pad_copy(lse, lp, (long long)d.B * d.heads, d.H0, d.W0, d.H, d.W, 4, true, st) != cudaSuccess) ok = false;
        lse = lp;
    }
    if (!ok) return BRA_ERR_CUDA;
    cudaError_t e = launch_backward(d, p->dtype, p->impl, Q, K, V, index, lce_w, lse, dO, pad_out(d, L, w, 4, dQ),
                                    pad_out(d, L, w, 5, dK), pad_out(d, L, w, 6, dV), d_lce_w, d_lce_b, w, L, st);
    if (e != cudaSuccess) return BRA_ERR_CUDA;
    crop_out(d, L, w, 4, dQ, st, &ok);
    crop_out(d, L, w, 5, dK, st, &ok);
    crop_out(d, L, w, 6, dV, st, &ok);
    return ok ? BRA_OK : BRA_ERR_CUDA;
}

bra_status bra_workspace_init(const bra_problem* p, void* ws, size_t ws_bytes, void* stream) {
    g_launches = 0;
    Dims d;
    bra_status s = make_dims(p, &d);
    if (s != BRA_OK) return s;
    WsLayout L;
    if ((s = check_ws(d, ws, ws_bytes, &L)) != BRA_OK) return s;
    char* w = static_cast<char*>(ws);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the status block (error words, barrier counters of the one-launch forward); the rest is written before it is read
    if (cudaMemsetAsync(w + L.status, 0, 256, st) != cudaSuccess) return BRA_ERR_CUDA;
    return BRA_OK;
}

bra_status bra_device_status(void* ws, void* stream) {
    if (!ws) return BRA_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t host[2] = {0, 0};           // code, detail
    if (cudaMemcpyAsync(host, ws, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return BRA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return BRA_ERR_CUDA;
    if (host[0] != 0) {
        // a kernel that gave up leaves its barrier counters as they were: clear the whole status block with
        // the error, so that the next call on this ws starts clean
        if (cudaMemsetAsync(ws, 0, 256, st) != cudaSuccess) return BRA_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return BRA_ERR_CUDA;
    }
    if (host[0] < 0 || host[0] > BRA_ERR_TIMEOUT) return BRA_ERR_CUDA;
    return static_cast<bra_status>(host[0]);
}

int32_t bra_last_launch_count(void) { return g_launches; }

const char* bra_status_string(bra_status s) {
    switch (s) {
        case BRA_OK: return "ok";
        case BRA_ERR_NULL: return "a required pointer is NULL";
        case BRA_ERR_SHAPE: return "bad shape: sizes must be positive, S must divide H and W, heads must divide C";
        case BRA_ERR_TOPK: return "topk must be in [1, S*S]";
        case BRA_ERR_DTYPE: return "dtype must be BRA_F32 or BRA_BF16";
        case BRA_ERR_ALIGN: return "pointer not aligned (tensors 16 bytes, workspace 256 bytes)";
        case BRA_ERR_WORKSPACE: return "workspace smaller than bra_workspace_bytes()";
        case BRA_ERR_UNSUPPORTED: return "no kernel in this build for this problem";
        case BRA_ERR_CUDA: return "a CUDA runtime call failed";
        case BRA_ERR_INDEX: return "routing index entry outside [0, S*S) (detected on the device)";
        case BRA_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case BRA_ERR_STATIC_LIMIT: return "problem larger than the built-in scratch of the no-allocation entry point";
    }
    return "unknown status";
}

int32_t bra_version(void) { return 200; }

}  // extern "C"
