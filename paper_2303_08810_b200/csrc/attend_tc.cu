// Routed token-to-token attention + LCE on the 5th-generation tensor cores
// (Eq. 6, Eq. 7 with Eq. 1): TMA streams the routed regions' K/V tiles by index
// straight into shared memory (K^g / V^g are never formed in HBM), tcgen05.mma
// computes S = Q K^T and O = P V with fp32 accumulators in tensor memory, the
// softmax runs in registers, and the 5x5 depthwise LCE of V is added from a
// shared-memory halo tile before the single store of O.
//
// Shape handled here: head dim 32, regions of 8 x 8 = 64 tokens, heads in pairs.
// One CTA owns (image b, query region i, head pair hp) = a 64-token x 64-channel
// tile of O.  The two heads are stacked into one 128-row MMA tile:
//     rows   0..63  = head A queries, rows 64..127 = head B queries
//     keys   0..63  = head A's routed region, keys 64..127 = head B's
// so S is 128 x 128 of which each row uses its own head's 64 columns (the
// diagonal blocks); P carries zeros in the off-diagonal blocks, which makes
// O = P [V_A; V_B] exact for both heads at once.
#include "bra_internal.h"
#include "sm100_ptx.cuh"

namespace bra {

using namespace ptx;

namespace tc {
constexpr int TOK = 64;          // tokens per region (8 x 8)
constexpr int RS = 8;            // region side in tokens
constexpr int HALO = RS + 4;     // 12: region plus the 2-token LCE border
constexpr int THREADS = 128;
constexpr int TMEM_COLS = 128;

// shared memory map (bytes, from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                       // [128 rows][64 B]  64B-swizzled, K-major
constexpr int OFF_K = OFF_Q + 8192;            // [128 keys][64 B]  64B-swizzled, K-major
constexpr int OFF_V = OFF_K + 8192;            // [128 keys][64 B]  64B-swizzled, MN-major (d contiguous)
constexpr int OFF_P = OFF_V + 8192;            // [2 chunks][128 rows][128 B] 128B-swizzled, K-major
constexpr int OFF_HALO = OFF_P + 32768;        // [12][12][64 ch] bf16, linear
constexpr int OFF_BAR = OFF_HALO + HALO * HALO * 128;   // 18432
constexpr int SMEM_BYTES = OFF_BAR + 64;
constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;  // slack for the manual 1024-byte alignment
}  // namespace tc

struct TcMaps {
    CUtensorMap q, k, v;     // box {32 ch, 8, 8, 1}, 64B swizzle
    CUtensorMap halo;        // V, box {64 ch, 12, 12, 1}, no swizzle, zero fill outside the map
};

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

__global__ void __launch_bounds__(tc::THREADS)
attend_tc_kernel(const __grid_constant__ TcMaps maps, const int32_t* __restrict__ index,
                 const float* __restrict__ lce_w, const float* __restrict__ lce_b,
                 __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
                 int32_t* __restrict__ status, Dims dm) {
    using namespace tc;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bar_q = reinterpret_cast<uint64_t*>(smem + OFF_BAR);        // Q tile + V halo landed
    uint64_t* bar_kv = bar_q + 1;                                         // K, V tiles of one routed region pair
    uint64_t* bar_mma = bar_q + 2;                                        // MMA group finished
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_q + 3);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pairs = dm.heads >> 1;
    const int hp = blockIdx.x % pairs;
    const int i = (blockIdx.x / pairs) % dm.R;
    const int b = blockIdx.x / (pairs * dm.R);
    const int y0 = (i / dm.S) * RS, x0 = (i % dm.S) * RS;
    const int c0 = hp * 64;                      // first channel of the pair
    const int hA = 2 * hp, hB = 2 * hp + 1;
    const int hiA = dm.heads_i == 1 ? 0 : hA, hiB = dm.heads_i == 1 ? 0 : hB;
    const int32_t* rowA = index + (((size_t)b * dm.heads_i + hiA) * dm.R + i) * dm.topk;
    const int32_t* rowB = index + (((size_t)b * dm.heads_i + hiB) * dm.R + i) * dm.topk;
    bool timed_out = false;

    if (tid == 0) {
        mbar_init(bar_q, 1);
        mbar_init(bar_kv, 1);
        mbar_init(bar_mma, 1);
        fence_mbar_init();
        prefetch_tmap(&maps.q); prefetch_tmap(&maps.k); prefetch_tmap(&maps.v); prefetch_tmap(&maps.halo);
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(tmem_slot, TMEM_COLS);
    // the off-diagonal blocks of P stay zero for the whole kernel:
    // chunk 0 (keys 0..63) rows 64..127 and chunk 1 (keys 64..127) rows 0..63
    {
        uint4 z = make_uint4(0, 0, 0, 0);
        uint8_t* zrow = smem + OFF_P + (tid < 64 ? 16384 + tid * 128 : (tid) * 128);
#pragma unroll
        for (int u = 0; u < 8; ++u) *reinterpret_cast<uint4*>(zrow + u * 16) = z;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    auto issue_kv = [&](int m) {     // leader only: stream the m-th routed regions of both heads
        int rA = rowA[m], rB = rowB[m];
        if (rA < 0 || rA >= dm.R) { record_error(status, BRA_ERR_INDEX, rA); rA = -1; }
        if (rB < 0 || rB >= dm.R) { record_error(status, BRA_ERR_INDEX, rB); rB = -1; }
        const int ra = rA < 0 ? 0 : rA, rb = rB < 0 ? 0 : rB;   // an invalid entry loads region 0, masked below
        mbar_expect_tx(bar_kv, 4 * 4096);
        tma_load_4d(smem + OFF_K, &maps.k, bar_kv, c0, (ra % dm.S) * RS, (ra / dm.S) * RS, b);
        tma_load_4d(smem + OFF_K + 4096, &maps.k, bar_kv, c0 + 32, (rb % dm.S) * RS, (rb / dm.S) * RS, b);
        tma_load_4d(smem + OFF_V, &maps.v, bar_kv, c0, (ra % dm.S) * RS, (ra / dm.S) * RS, b);
        tma_load_4d(smem + OFF_V + 4096, &maps.v, bar_kv, c0 + 32, (rb % dm.S) * RS, (rb / dm.S) * RS, b);
    };

    if (tid == 0) {
        const uint32_t bytes = 8192 + (dm.lce ? HALO * HALO * 128 : 0);
        mbar_expect_tx(bar_q, bytes);
        tma_load_4d(smem + OFF_Q, &maps.q, bar_q, c0, x0, y0, b);
        tma_load_4d(smem + OFF_Q + 4096, &maps.q, bar_q, c0 + 32, x0, y0, b);
        if (dm.lce) tma_load_4d(smem + OFF_HALO, &maps.halo, bar_q, c0, x0 - 2, y0 - 2, b);
        issue_kv(0);
    }

    // ---- attention: thread = one row of the 128-row tile -------------------------
    const int head_half = tid >> 6;                // 0: head A, 1: head B
    const int tq = tid & 63;                       // query token inside the region
    const float sl2 = dm.scale * 1.4426950408889634f;
    float m_run = -INFINITY, l_run = 0.f;
    float o_acc[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) o_acc[c] = 0.f;
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
    uint32_t mma_phase = 0;
    constexpr uint32_t IDESC_S = umma_idesc_bf16(128, 128, false, false);
    constexpr uint32_t IDESC_O = umma_idesc_bf16(128, 32, false, true);

    for (int m = 0; m < dm.topk; ++m) {
        if (tid == 0) {
            if (m == 0 && !mbar_wait(bar_q, 0)) timed_out = true;
            if (!mbar_wait(bar_kv, m & 1)) timed_out = true;
            tc_fence_after_sync();
            const uint32_t qa = smem_u32(smem + OFF_Q), ka = smem_u32(smem + OFF_K);
#pragma unroll
            for (int ks = 0; ks < 2; ++ks)         // d = 32 = 2 k-steps of 16
                umma_ss(tmem, umma_smem_desc(qa + ks * 32, 16, 512, 4), umma_smem_desc(ka + ks * 32, 16, 512, 4),
                        IDESC_S, ks);
            umma_commit(bar_mma);
        }
        if (!mbar_wait(bar_mma, mma_phase)) timed_out = true;
        mma_phase ^= 1;
        tc_fence_after_sync();
        const int r_mine = head_half ? rowB[m] : rowA[m];
        const bool valid = r_mine >= 0 && r_mine < dm.R;

        uint32_t sraw[64];
        tmem_ld_32x32b_x32(lane_base + head_half * 64, sraw);
        tmem_ld_32x32b_x32(lane_base + head_half * 64 + 32, sraw + 32);
        tmem_ld_wait();
        float mx = m_run;
        if (valid) {
#pragma unroll
            for (int j = 0; j < 64; ++j) mx = fmaxf(mx, __uint_as_float(sraw[j]) * sl2);
        }
        const float corr = (mx == -INFINITY) ? 1.f : ex2f(m_run - mx);
        const float mneg = (mx == -INFINITY) ? 0.f : -mx;
        float sum = 0.f;
        uint32_t pk[32];
#pragma unroll
        for (int j = 0; j < 64; j += 2) {
            float p0 = valid ? ex2f(fmaf(__uint_as_float(sraw[j]), sl2, mneg)) : 0.f;
            float p1 = valid ? ex2f(fmaf(__uint_as_float(sraw[j + 1]), sl2, mneg)) : 0.f;
            sum += p0 + p1;
            pk[j >> 1] = pack_bf16(p0, p1);
        }
        l_run = l_run * corr + sum;
        m_run = mx;
        {   // P row -> its diagonal block: chunk = head_half, row = tid, 128B swizzle
            uint8_t* prow = smem + OFF_P + head_half * 16384 + tid * 128;
#pragma unroll
            for (int u = 0; u < 8; ++u)
                *reinterpret_cast<uint4*>(prow + ((u ^ (tid & 7)) << 4)) =
                    make_uint4(pk[4 * u], pk[4 * u + 1], pk[4 * u + 2], pk[4 * u + 3]);
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t pa = smem_u32(smem + OFF_P), va = smem_u32(smem + OFF_V);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)         // 128 keys = 8 k-steps of 16
                umma_ss(tmem, umma_smem_desc(pa + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024, 2),
                        umma_smem_desc(va + ks * 1024, 16, 512, 4), IDESC_O, ks);
            umma_commit(bar_mma);
        }
        if (!mbar_wait(bar_mma, mma_phase)) timed_out = true;
        mma_phase ^= 1;
        tc_fence_after_sync();
        uint32_t oraw[32];
        tmem_ld_32x32b_x32(lane_base, oraw);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 32; ++c) o_acc[c] = fmaf(o_acc[c], corr, __uint_as_float(oraw[c]));
        tc_fence_before_sync();
        __syncthreads();                           // S/O columns and the K/V tiles are free again
        if (tid == 0 && m + 1 < dm.topk) issue_kv(m + 1);
    }

    // ---- epilogue: normalise, stage O^att as fp32 [64 tokens][64 ch] over the P buffer ----
    // LCE weights of this thread's channel pair, kept in registers (lane = channel pair);
    // issued here so the loads fly while O^att is staged
    float w0[25], w1[25];
    if (dm.lce) {
        const float* wp = lce_w + (size_t)(c0 + 2 * lane) * 25;
#pragma unroll
        for (int k = 0; k < 25; ++k) { w0[k] = __ldg(wp + k); w1[k] = __ldg(wp + 25 + k); }
    }
    const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
    float* stage = reinterpret_cast<float*>(smem + OFF_P);
    {
        uint8_t* srow = reinterpret_cast<uint8_t*>(stage) + tq * 256;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int chunk = head_half * 8 + u;
            *reinterpret_cast<float4*>(srow + ((chunk ^ (tq & 7)) << 4)) =
                make_float4(o_acc[4 * u] * inv, o_acc[4 * u + 1] * inv, o_acc[4 * u + 2] * inv, o_acc[4 * u + 3] * inv);
        }
    }
    if (lse) {
        const int hh = head_half ? hB : hA;
        lse[((size_t)b * dm.heads + hh) * dm.N + (size_t)(y0 + tq / RS) * dm.W + x0 + tq % RS] =
            (m_run + log2f(l_run)) * 0.6931471805599453f;
    }
    if (dm.lce && tid != 0 && !mbar_wait(bar_q, 0)) timed_out = true;    // halo visible to every reader
    __syncthreads();

    // ---- LCE + store: warp = 2 columns of the region, lane = channel pair -----------
    {
        const int xl0 = 2 * warp;
        float a0[8][2], a1[8][2];
#pragma unroll
        for (int y = 0; y < 8; ++y)
#pragma unroll
            for (int xx = 0; xx < 2; ++xx) { a0[y][xx] = 0.f; a1[y][xx] = 0.f; }
        if (dm.lce) {
            const uint32_t* halo = reinterpret_cast<const uint32_t*>(smem + OFF_HALO) + lane;
#pragma unroll
            for (int yy = 0; yy < HALO; ++yy) {
                float v0[6], v1[6];
#pragma unroll
                for (int xx = 0; xx < 6; ++xx) {
                    const uint32_t u = halo[(yy * HALO + xl0 + xx) * 32];
                    v0[xx] = __uint_as_float(u << 16);
                    v1[xx] = __uint_as_float(u & 0xffff0000u);
                }
#pragma unroll
                for (int ti = 0; ti < 5; ++ti) {
                    const int y = yy - ti;             // output row fed by this input row through tap row ti
                    if (y < 0 || y >= 8) continue;
#pragma unroll
                    for (int xx = 0; xx < 2; ++xx)
#pragma unroll
                        for (int tj = 0; tj < 5; ++tj) {
                            a0[y][xx] = fmaf(w0[ti * 5 + tj], v0[xx + tj], a0[y][xx]);
                            a1[y][xx] = fmaf(w1[ti * 5 + tj], v1[xx + tj], a1[y][xx]);
                        }
                }
            }
            if (lce_b) {
                const float b0 = __ldg(lce_b + c0 + 2 * lane), b1 = __ldg(lce_b + c0 + 2 * lane + 1);
#pragma unroll
                for (int y = 0; y < 8; ++y)
#pragma unroll
                    for (int xx = 0; xx < 2; ++xx) { a0[y][xx] += b0; a1[y][xx] += b1; }
            }
        }
        uint32_t* out = reinterpret_cast<uint32_t*>(O) + ((((size_t)b * dm.H + y0) * dm.W + x0) * dm.C + c0) / 2 + lane;
#pragma unroll
        for (int y = 0; y < 8; ++y)
#pragma unroll
            for (int xx = 0; xx < 2; ++xx) {
                const int t = y * RS + xl0 + xx;
                const float2 att = *reinterpret_cast<const float2*>(
                    reinterpret_cast<const uint8_t*>(stage) + t * 256 + (((lane >> 1) ^ (t & 7)) << 4) + (lane & 1) * 8);
                out[((size_t)y * dm.W + xl0 + xx) * (dm.C / 2)] = pack_bf16(att.x + a0[y][xx], att.y + a1[y][xx]);
            }
    }

    if (timed_out) record_error(status, BRA_ERR_TIMEOUT, blockIdx.x);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [B,H,W,C] bf16 tensor, box {bc, bx, by, 1}
static bool make_map(CUtensorMap* m, const void* base, const Dims& d, uint32_t bc, uint32_t bx, uint32_t by,
                     CUtensorMapSwizzle sw) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)d.C, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.B};
    cuuint64_t strides[3] = {(cuuint64_t)d.C * 2, (cuuint64_t)d.W * d.C * 2, (cuuint64_t)d.H * d.W * d.C * 2};
    cuuint32_t box[4] = {bc, bx, by, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool attend_tc_supported(const Dims& d, int dtype) {
    return dtype == BRA_BF16 && d.d == 32 && d.heads % 2 == 0 && d.hs == tc::RS && d.ws == tc::RS;
}

cudaError_t launch_attend_tc(const Dims& d, const void* Q, const void* K, const void* V,
                             const int32_t* index, const float* lce_w, const float* lce_b,
                             void* O, float* lse, int32_t* status, cudaStream_t st) {
    TcMaps maps;
    if (!make_map(&maps.q, Q, d, 32, tc::RS, tc::RS, CU_TENSOR_MAP_SWIZZLE_64B) ||
        !make_map(&maps.k, K, d, 32, tc::RS, tc::RS, CU_TENSOR_MAP_SWIZZLE_64B) ||
        !make_map(&maps.v, V, d, 32, tc::RS, tc::RS, CU_TENSOR_MAP_SWIZZLE_64B) ||
        !make_map(&maps.halo, V, d, 64, tc::HALO, tc::HALO, CU_TENSOR_MAP_SWIZZLE_NONE))
        return cudaErrorInvalidValue;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_ALLOC);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const unsigned grid = (unsigned)d.B * d.R * (d.heads / 2);
    attend_tc_kernel<<<grid, tc::THREADS, tc::SMEM_ALLOC, st>>>(
        maps, index, lce_w, lce_b, static_cast<__nv_bfloat16*>(O), lse, status, d);
    count_launch();
    return cudaGetLastError();
}

}  // namespace bra
