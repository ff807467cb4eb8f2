// Routed token-to-token attention + LCE on the 5th-generation tensor cores
// (Eq. 6, Eq. 7 with Eq. 1).
//
// Shape handled here: head dim 32, regions of 8 x 8 = 64 tokens, heads in pairs.
// A tile is (image b, query region i, head pair hp) = 64 tokens x 64 channels of O.
// The two heads are stacked into one 128-row MMA tile:
//     rows   0..63  = head A queries, rows 64..127 = head B queries
//     keys   0..63  = head A's routed region, keys 64..127 = head B's
// S = Q K^T is 128 x 128 of which each row uses its own head's 64 columns.  For O = P V
// the two heads share the key axis instead: P is 128 x 64 (row r, key j of r's own head)
// and V is 64 x 64 with key j's row = (head A's channels of token j of A's region | head
// B's channels of token j of B's region); each row then keeps its own head's 32 columns.
//
// Small CTAs (128 threads, ~51 KB of shared memory, 128 TMEM columns), four per SM,
// each walking its own tiles start to finish; the SM overlaps the CTAs' phases.
// Measured on this shape, that beats one large warp-specialised CTA per SM: the work
// per tile is too small to pay for hand-offs between specialised warps.  Per tile:
//   1. all threads: 16-byte cp.async copies of the Q tile, of the K and V tiles of the
//      routed regions (K^g / V^g are never formed in HBM: the routing index only picks
//      the source addresses) and of the 12 x 12 V halo, written in the 64-byte swizzled
//      layout the MMA descriptors name.  Issued one tile ahead, around the LCE of the
//      tile in hand.  (Many small copies in flight reach a multiple of the bandwidth
//      that one bulk tensor copy per 4-18 KB box gives at these box sizes.)
//   2. one thread: tcgen05.mma S = Q K^T into TMEM (fp32)
//   3. thread = row: softmax; P (bf16 pairs) overwrites S in TMEM columns 0..63
//   4. one thread: tcgen05.mma O = P V with P read from TMEM; O lands in columns 64..95
//   5. thread = row: normalised O^att to an fp32 staging tile
//   6. warp = 2 columns of the region, lane = channel pair: LCE, the 5x5 depthwise
//      correlation of V from the halo tile with the weights in registers, + O^att, one
//      bf16 store of O.
// Hot loops are kept rolled and short (straight-line per-tile code was bound by
// instruction fetch).  Every wait on an MMA is bounded.
#include "bra_internal.h"
#include "sm100_ptx.cuh"
#ifdef BRA_TRACE
#include <cstdio>
#endif

namespace bra {

using namespace ptx;

namespace tc {
constexpr int RS = 8;            // region side in tokens
constexpr int HALO = RS + 4;     // 12: region plus the 2-token LCE border
constexpr int THREADS = 128;
constexpr int KCAP = 64;         // largest topk
constexpr int TMEM_COLS = 128;   // S [0,128) fp32; then P [0,32) bf16 pairs + O [64,128)
constexpr int TM_O = 64;
constexpr int HALO_BYTES = HALO * HALO * 128;            // 18432
// shared memory map (bytes, from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                                 // [128 rows][64 B]  64B swizzle, K-major
constexpr int OFF_ST = 0;                                // [64 tokens][64 ch] fp32: over Q, + 8 KB of its own
constexpr int OFF_K = 16384;                             // [128 keys][64 B]  64B swizzle, K-major (buffer 0)
constexpr int OFF_V = 24576;                             // [64 keys][128 B]  128B swizzle, MN-major (buffer 0)
constexpr int OFF_HALO = 32768;                          // [12][12][64 ch] bf16, linear
constexpr int OFF_BAR = OFF_HALO + HALO_BYTES;           // 51200: two mbarriers, tmem slot
constexpr int OFF_KV1 = 52224;                           // topk > 1 only: K buffer 1 (8 KB), V buffer 1 (8 KB)
constexpr int SMEM_K1 = OFF_BAR + 64 + 1024;             // + slack for the manual 1024-byte alignment
constexpr int SMEM_KN = OFF_KV1 + 16384 + 1024;
static_assert(OFF_KV1 % 1024 == 0 && OFF_KV1 >= OFF_BAR + 64, "buffer 1 placement");
constexpr uint32_t POLL_LIMIT = 4000000u;
}  // namespace tc

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// Optional timeline of CTA 0 (compile with -DBRA_TRACE): clock64() stamps of the phases,
// [tile][event], read back with bra_debug_read_trace().  Off in normal builds.
#ifdef BRA_TRACE
__device__ long long g_trace[32 * 8];
#define BRA_TR(tile, ev)                                                                       \
    do {                                                                                       \
        if (threadIdx.x == 0 && blockIdx.x == 0 && (tile) < 32) g_trace[(tile) * 8 + (ev)] = clock64(); \
    } while (0)
#else
#define BRA_TR(tile, ev) do { } while (0)
#endif

struct TileCoord { int b, i, hp, y0, x0, c0; };
// Walks tiles T, T + stride, ... (T = (b * R + i) * pairs + hp) with adds and carries only.
struct TileWalker {
    int pairs, R, S, inv_s;            // inv_s: i / S == (i * inv_s) >> 20 for i < 4096
    int d_hp, d_i, d_b;                // stride split into (hp, i, b) digits
    int hp, i, b;
    __device__ __forceinline__ void init(int T, int stride, const Dims& dm) {
        pairs = dm.heads >> 1; R = dm.R; S = dm.S;
        inv_s = (1 << 20) / S + 1;
        hp = T % pairs; i = (T / pairs) % R; b = T / (pairs * R);
        d_hp = stride % pairs; d_i = (stride / pairs) % R; d_b = stride / (pairs * R);
    }
    __device__ __forceinline__ void next() {
        hp += d_hp;
        int carry = hp >= pairs;
        hp -= carry ? pairs : 0;
        i += d_i + carry;
        carry = i >= R;
        i -= carry ? R : 0;
        b += d_b + carry;
    }
    __device__ __forceinline__ TileCoord coord() const {
        TileCoord t;
        t.b = b; t.i = i; t.hp = hp;
        const int ry = (i * inv_s) >> 20;
        t.y0 = ry * tc::RS;
        t.x0 = (i - ry * S) * tc::RS;
        t.c0 = hp * 64;
        return t;
    }
};

// K1: topk == 1 (one routed step per tile: no running maximum, no rescaling of O, one K/V buffer).
template <bool K1>
__global__ void __launch_bounds__(tc::THREADS, K1 ? 4 : 3)
attend_tc_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                 const __nv_bfloat16* __restrict__ Vg, const int32_t* index,
                 const float* __restrict__ lce_w, const float* __restrict__ lce_b,
                 __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
                 int32_t* __restrict__ status, Dims dm, int num_tiles) {
    using namespace tc;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bar_s = reinterpret_cast<uint64_t*>(smem + OFF_BAR);       // S landed in TMEM
    uint64_t* bar_o = bar_s + 1;                                         // O landed in TMEM
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_s + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int k = K1 ? 1 : dm.topk;
    const int my_tiles = (num_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (tid == 0) {
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    TileWalker walk;
    walk.init(blockIdx.x, gridDim.x, dm);

    // ---- loader mapping: thread copies 16-byte chunk c of the 128-byte channel row (both
    // heads) of token column tx, in token rows lrow..lrow+3 of a region: a warp covers 512
    // contiguous bytes per instruction.  Chunks 0-3 are head A, 4-7 head B; inside a head's
    // [token][64 B] tile the chunk index is xor-ed with (token >> 1) & 3 (64-byte swizzle).
    const int c = tid & 7, tx = (tid >> 3) & 7, lrow = (tid >> 6) * 4;
    const int lhead = c >> 2;
    const uint32_t tile_off = lhead * 4096 + (lrow * 8 + tx) * 64 + (((c & 3) ^ ((tx >> 1) & 3)) << 4);
    // V: [key][128 B] with both heads side by side, 16-byte chunk index xor-ed with key & 7 (= tx)
    const uint32_t v_off = (lrow * 8 + tx) * 128 + ((c ^ tx) << 4);
    const size_t row_bytes = (size_t)dm.W * dm.C * 2;
    const uint32_t sm_base = smem_u32(smem);
    const uint8_t* Qb = reinterpret_cast<const uint8_t*>(Qg);
    const uint8_t* Kb = reinterpret_cast<const uint8_t*>(Kg);
    const uint8_t* Vb = reinterpret_cast<const uint8_t*>(Vg);

    // ---- softmax mapping: thread = row of the stacked tile = TMEM lane
    const int head_half = tid >> 6;                    // 0: head A, 1: head B
    const int tq = tid & 63;                           // query token inside the region
    const uint32_t tg = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t s_addr = tg + head_half * 64;       // this row's 64 scores
    const uint32_t p_addr = tg;                        // this row's 64 probabilities (bf16 pairs)
    const uint32_t o_addr = tg + TM_O + head_half * 32;   // this row's 32 channels of O
    const float sl2 = dm.scale * 1.4426950408889634f;
    // ---- LCE mapping: warp = 2 columns of the region, lane = channel pair
    const int xl0 = 2 * warp;
    float2 wv[25];
#pragma unroll
    for (int q = 0; q < 25; ++q) wv[q] = make_float2(0.f, 0.f);
    float2 bias2 = make_float2(0.f, 0.f);
    int hp_loaded = -1;

    constexpr uint32_t IDESC_S = umma_idesc_bf16(128, 128, false, false);
    constexpr uint32_t IDESC_O = umma_idesc_bf16(128, 64, false, true);

    // routing entries (head A, head B) of a unit = (tile, routed step); -1: out of range.  The index may
    // come from a kernel this one overlaps (programmatic dependent launch): coherent loads after pdl_wait(),
    // never the read-only path, whose loads the compiler may move above the wait
    auto read_entries = [&](const TileCoord& t, int m) -> int2 {
        const int hA = 2 * t.hp, hB = hA + 1;
        const int hiA = dm.heads_i == 1 ? 0 : hA, hiB = dm.heads_i == 1 ? 0 : hB;
        int ra = __ldcg(index + (((size_t)t.b * dm.heads_i + hiA) * dm.R + t.i) * dm.topk + m);
        int rb = __ldcg(index + (((size_t)t.b * dm.heads_i + hiB) * dm.R + t.i) * dm.topk + m);
        if (ra < 0 || ra >= dm.R) { record_error(status, BRA_ERR_INDEX, ra); ra = -1; }
        if (rb < 0 || rb >= dm.R) { record_error(status, BRA_ERR_INDEX, rb); rb = -1; }
        return make_int2(ra, rb);
    };
    auto load_kv = [&](const TileCoord& t, int2 ent, int buf) {
        int r = lhead ? ent.y : ent.x;
        r = r < 0 ? 0 : r;                  // an invalid entry loads region 0; its P is zero
        const int ry = (r * walk.inv_s) >> 20, rx = r - ry * dm.S;
        const size_t off = (size_t)t.b * dm.H * row_bytes + (size_t)(ry * RS + lrow) * row_bytes +
                           (size_t)(rx * RS + tx) * dm.C * 2 + (size_t)t.c0 * 2 + c * 16;
        const uint32_t kd = sm_base + (buf ? OFF_KV1 : OFF_K) + tile_off;
        const uint32_t vd = sm_base + (buf ? OFF_KV1 + 8192 : OFF_V) + v_off;
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async_16(kd + i * 512, Kb + off + i * row_bytes, 16);
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async_16(vd + i * 1024, Vb + off + i * row_bytes, 16);
    };
    // halo chunk i of this thread is token pos = (tid >> 3) + 16 i of the 12 x 12 tile: its byte
    // offset from the tile's first token, and which map edges would put it outside
    int32_t h_off[9];
    uint32_t m_top = 0, m_bot = 0, m_left = 0, m_right = 0;
#pragma unroll
    for (int i = 0; i < 9; ++i) {
        const int pos = (tid >> 3) + 16 * i;
        const int hy = pos / HALO, hx = pos - hy * HALO;
        h_off[i] = (hy - 2) * (int32_t)row_bytes + (hx - 2) * dm.C * 2;
        m_top |= (hy < 2) << i;  m_bot |= (hy >= HALO - 2) << i;
        m_left |= (hx < 2) << i; m_right |= (hx >= HALO - 2) << i;
    }
    auto load_q_halo = [&](const TileCoord& t) {
        const size_t img = (size_t)t.b * dm.H * row_bytes;
        const size_t in_row = (size_t)t.c0 * 2 + c * 16;
        const uint8_t* src = Qb + img + (size_t)(t.y0 + lrow) * row_bytes + (size_t)(t.x0 + tx) * dm.C * 2 + in_row;
        const uint32_t dst = sm_base + OFF_Q + tile_off;
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async_16(dst + i * 512, src + i * row_bytes, 16);
        if (dm.lce) {
            // 12 x 12 tokens x 128 B around the region, zeros outside the map; 9 chunks per thread
            const uint32_t hd = sm_base + OFF_HALO + tid * 16;
            const uint8_t* org = Vb + img + (size_t)t.y0 * row_bytes + (size_t)t.x0 * dm.C * 2 + in_row;
            const uint32_t outside = (t.y0 == 0 ? m_top : 0u) | (t.y0 + RS == dm.H ? m_bot : 0u) |
                                     (t.x0 == 0 ? m_left : 0u) | (t.x0 + RS == dm.W ? m_right : 0u);
#pragma unroll
            for (int i = 0; i < 9; ++i) {
                const bool inb = !((outside >> i) & 1u);
                cp_async_16(hd + i * 2048, inb ? org + h_off[i] : Vb, inb ? 16u : 0u);
            }
        }
    };

    bool ok = true;
    uint32_t n_s = 0, n_o = 0;              // uses of bar_s / bar_o so far (phase parity)
    TileCoord t = walk.coord();
    // Q and the V halo are inputs of the call: their copies (and everything above) overlap the tail of
    // the kernel before (routing, in bra_forward); only the routing index has to wait for it
    if (my_tiles > 0) load_q_halo(t);
    pdl_wait();
    int2 ent = read_entries(t, 0);          // entries of the unit whose K/V are being loaded
    if (my_tiles > 0) load_kv(t, ent, 0);
    cp_async_commit();

    for (int n = 0; n < my_tiles && ok; ++n) {
        if (dm.lce && t.hp != hp_loaded) {
            const float* wp = lce_w + (size_t)(t.c0 + 2 * lane) * 25;
#pragma unroll
            for (int q = 0; q < 25; ++q) wv[q] = make_float2(__ldg(wp + q), __ldg(wp + 25 + q));
            if (lce_b) bias2 = make_float2(__ldg(lce_b + t.c0 + 2 * lane), __ldg(lce_b + t.c0 + 2 * lane + 1));
            hp_loaded = t.hp;
        }
        const bool has_next = n + 1 < my_tiles;
        if (has_next) walk.next();
        const TileCoord tn = has_next ? walk.coord() : t;

        float m_run = -INFINITY, l_run = 0.f;
        float o_acc[32];
#pragma unroll
        for (int q = 0; q < 32; ++q) o_acc[q] = 0.f;
        BRA_TR(n, 0);
        for (int m = 0; m < k; ++m) {
            const int buf = K1 ? 0 : (m & 1);
            const int2 ent_cur = ent;
            // ---- the copies of this step have landed; make them visible to the tensor core ----
            cp_async_wait<0>();
            fence_proxy_async_smem();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after_sync();
                const uint32_t qa = sm_base + OFF_Q;
                const uint32_t ka = sm_base + (buf ? OFF_KV1 : OFF_K);
#pragma unroll
                for (int ks = 0; ks < 2; ++ks)         // d = 32 = 2 k-steps of 16
                    umma_ss(tmem, umma_smem_desc(qa + ks * 32, 16, 512, 4),
                            umma_smem_desc(ka + ks * 32, 16, 512, 4), IDESC_S, ks);
                umma_commit(bar_s);
            }
            // ---- next routed step of this tile: K/V into the other buffer (its MMAs are done) ----
            if (!K1 && m + 1 < k) {
                ent = read_entries(t, m + 1);
                load_kv(t, ent, buf ^ 1);
                cp_async_commit();
            } else if (has_next) {
                ent = read_entries(tn, 0);             // in flight during the softmax
            }
            const bool valid = (head_half ? ent_cur.y : ent_cur.x) >= 0;
            BRA_TR(n, 1);
            if (warp == 0) ok = mbar_wait(bar_s, n_s & 1, POLL_LIMIT);   // one warp polls, the rest sleep at the barrier
            ++n_s;
            if (!__syncthreads_and(ok)) { ok = false; break; }
            tc_fence_after_sync();
            BRA_TR(n, 2);
            // pass 1: row maximum
            float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll 1
            for (int cc = 0; cc < 64; cc += 16) {
                uint32_t r[16];
                tmem_ld_32x32b_x16(s_addr + cc, r);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 16; q += 4) {
                    m0 = fmax3(m0, __uint_as_float(r[q]), __uint_as_float(r[q + 1]));
                    m1 = fmax3(m1, __uint_as_float(r[q + 2]), __uint_as_float(r[q + 3]));
                }
            }
            float mx = m_run;
            if (valid) mx = fmaxf(mx, fmaxf(m0, m1) * sl2);               // sl2 > 0
            const float corr = (mx == -INFINITY) ? 1.f : ex2f(m_run - mx);
            const float mneg = (mx == -INFINITY) ? 0.f : -mx;
            m_run = mx;
            // pass 2: P = exp2(S * scale * log2 e - max), bf16 pairs written over the columns
            // of S already consumed (column j of P never outruns column 2j of S); row sum
            const float2 sl2v = make_float2(sl2, sl2), mnegv = make_float2(mneg, mneg);
            float2 sum2 = make_float2(0.f, 0.f);
#pragma unroll 1
            for (int cc = 0; cc < 64; cc += 16) {
                uint32_t r[16], pk[8];
                tmem_ld_32x32b_x16(s_addr + cc, r);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 16; q += 2) {
                    const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[q]), __uint_as_float(r[q + 1])), sl2v, mnegv);
                    const float2 pe = make_float2(valid ? ex2f(a.x) : 0.f, valid ? ex2f(a.y) : 0.f);
                    sum2 = __fadd2_rn(sum2, pe);
                    pk[q >> 1] = pack_bf16(pe.x, pe.y);
                }
                tmem_st_32x32b_x8(p_addr + (cc >> 1), pk);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncthreads();
            BRA_TR(n, 3);
            if (tid == 0) {
                tc_fence_after_sync();
                const uint64_t vd = umma_smem_desc(sm_base + (buf ? OFF_KV1 + 8192 : OFF_V), 16, 1024, 2);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)         // 64 keys = 4 k-steps of 16 (2048 B of V each)
                    umma_ts(tmem + TM_O, tmem + ks * 8, vd + (uint64_t)(ks * 128), IDESC_O, ks);
                umma_commit(bar_o);
            }
            if (warp == 0) ok = mbar_wait(bar_o, n_o & 1, POLL_LIMIT);
            ++n_o;
            if (!__syncthreads_and(ok)) { ok = false; break; }
            tc_fence_after_sync();
            BRA_TR(n, 4);
            uint32_t oraw[32];
            tmem_ld_32x32b_x32(o_addr, oraw);
            tmem_ld_wait();
            tc_fence_before_sync();
            if (K1) {
                l_run = sum2.x + sum2.y;
#pragma unroll
                for (int q = 0; q < 32; ++q) o_acc[q] = __uint_as_float(oraw[q]);
            } else {
                l_run = fmaf(l_run, corr, sum2.x + sum2.y);
#pragma unroll
                for (int q = 0; q < 32; ++q) o_acc[q] = fmaf(o_acc[q], corr, __uint_as_float(oraw[q]));
            }
        }
        if (!ok) break;

        // ---- normalise, stage O^att as fp32 [64 tokens][64 ch] (16-byte units xor-swizzled) ----
        {
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            const uint32_t srow = sm_base + OFF_ST + tq * 256;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int chunk = head_half * 8 + q;
                sts_f32x4(srow + ((chunk ^ (tq & 7)) << 4),
                          o_acc[4 * q] * inv, o_acc[4 * q + 1] * inv, o_acc[4 * q + 2] * inv, o_acc[4 * q + 3] * inv);
            }
            if (lse)
                lse[((size_t)t.b * dm.heads + 2 * t.hp + head_half) * dm.N + (size_t)(t.y0 + tq / RS) * dm.W + t.x0 + tq % RS] =
                    (m_run + log2f(l_run)) * 0.6931471805599453f;
        }
        // next tile's K / V (buffer 0 is free: all MMAs of this tile are done)
        if (has_next) load_kv(tn, ent, 0);
        cp_async_commit();
        __syncthreads();
        BRA_TR(n, 5);

        // ---- LCE + store ----
        // Input row yy of the halo feeds output rows yy - ti through tap row ti.  Fully unrolled:
        // the 8 x 2 output sums of this thread's channel pair sit in registers under fixed names.
        {
            const uint32_t halo = sm_base + OFF_HALO + (xl0 * 32 + lane) * 4;
            const uint32_t stage = sm_base + OFF_ST + xl0 * 256 + (lane & 1) * 8;
            uint32_t* out = reinterpret_cast<uint32_t*>(O) +
                            ((((size_t)t.b * dm.H + t.y0) * dm.W + t.x0 + xl0) * dm.C + t.c0) / 2 + lane;
            const size_t out_row = (size_t)dm.W * (dm.C / 2);
            float2 acc[8][2];
#pragma unroll
            for (int y = 0; y < 8; ++y) { acc[y][0] = bias2; acc[y][1] = bias2; }
            if (dm.lce) {
#pragma unroll
                for (int yy = 0; yy < HALO; ++yy) {
                    float2 v[6];
#pragma unroll
                    for (int xx = 0; xx < 6; ++xx) {
                        const uint32_t w = lds_u32(halo + (yy * HALO + xx) * 128);
                        v[xx] = make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
                    }
                    // tap column outermost: consecutive FMAs go to different sums
#pragma unroll
                    for (int tj = 0; tj < 5; ++tj)
#pragma unroll
                        for (int ti = 0; ti < 5; ++ti) {
                            const int y = yy - ti;
                            if (y < 0 || y >= 8) continue;
#pragma unroll
                            for (int xx = 0; xx < 2; ++xx)
                                acc[y][xx] = __ffma2_rn(wv[ti * 5 + tj], v[xx + tj], acc[y][xx]);
                        }
                }
            }
            // staging token tk = y * 8 + xl0 + xx: its 16-byte unit index is xor-ed with tk & 7
            const uint32_t sw0 = (((lane >> 1) ^ (xl0 & 7)) << 4), sw1 = (((lane >> 1) ^ ((xl0 + 1) & 7)) << 4);
#pragma unroll
            for (int y = 0; y < 8; ++y) {
#pragma unroll
                for (int xx = 0; xx < 2; ++xx) {
                    const float2 att = lds_f32x2(stage + (y * RS + xx) * 256 + (xx ? sw1 : sw0));
                    const float2 r = __fadd2_rn(att, acc[y][xx]);
                    out[xx * (dm.C / 2)] = pack_bf16(r.x, r.y);
                }
                out += out_row;
            }
        }
        __syncthreads();                    // staging tile (over Q) and halo are free
        BRA_TR(n, 6);
        if (has_next) load_q_halo(tn);
        cp_async_commit();
        t = tn;
    }

    // ---- teardown: nothing in flight, TMEM returned ----
    cp_async_wait<0>();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && !ok) record_error(status, BRA_ERR_TIMEOUT, blockIdx.x);
    if (warp == 0) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

// ------------------------------------------------------------------ host side
static int sm_count() {
    static int n[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
    if (!n[dev] && cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n[dev] = 1;
    return n[dev] > 0 ? n[dev] : 1;
}

bool attend_tc_supported(const Dims& d, int dtype) {
    return dtype == BRA_BF16 && d.d == 32 && d.heads % 2 == 0 && d.hs == tc::RS && d.ws == tc::RS &&
           d.topk <= tc::KCAP && (long long)d.B * d.R * (d.heads / 2) < (1ll << 30) &&
           (long long)d.W * d.C * 2 * tc::HALO < (1ll << 31) && d.R <= 4096;
}

cudaError_t launch_attend_tc(const Dims& d, const void* Q, const void* K, const void* V,
                             const int32_t* index, const float* lce_w, const float* lce_b,
                             void* O, float* lse, int32_t* status, cudaStream_t st) {
    static PerDeviceMax attr_set;
    if (attr_set.raise(1)) {
        cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_K1);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(attend_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_KN);
        if (e != cudaSuccess) return e;
        // several CTAs per SM: ask for the largest shared-memory carve-out
        e = cudaFuncSetAttribute(attend_tc_kernel<true>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(attend_tc_kernel<false>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
#ifdef BRA_TRACE
        int occ1 = 0, occn = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ1, attend_tc_kernel<true>, tc::THREADS, tc::SMEM_K1);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occn, attend_tc_kernel<false>, tc::THREADS, tc::SMEM_KN);
        printf("attend_tc occupancy: K1 %d CTAs/SM, general %d CTAs/SM\n", occ1, occn);
        cudaFuncAttributes fa;
        cudaFuncGetAttributes(&fa, attend_tc_kernel<true>);
        int smsm = 0, regs = 0;
        cudaDeviceGetAttribute(&smsm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, 0);
        cudaDeviceGetAttribute(&regs, cudaDevAttrMaxRegistersPerMultiprocessor, 0);
        printf("regs %d static smem %zu maxdyn %d carveout %d | SM smem %d regs %d\n", fa.numRegs, fa.sharedSizeBytes,
               fa.maxDynamicSharedSizeBytes, fa.preferredShmemCarveout, smsm, regs);
        for (int sz : {0, 16384, 32768, 49152, 52288, 60000}) {
            int o = 0;
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, attend_tc_kernel<true>, tc::THREADS, sz);
            printf("  dyn smem %d -> %d CTAs/SM\n", sz, o);
        }
#endif
    }
    const int tiles = d.B * d.R * (d.heads / 2);
    const int resident = sm_count() * (d.topk == 1 ? 4 : 3);
    const unsigned grid = (unsigned)(tiles < resident ? tiles : resident);
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(Q);
    const __nv_bfloat16* k = static_cast<const __nv_bfloat16*>(K);
    const __nv_bfloat16* v = static_cast<const __nv_bfloat16*>(V);
    const bool pdl = take_after_own_kernel();
    __nv_bfloat16* o = static_cast<__nv_bfloat16*>(O);
    cudaError_t e;
    if (d.topk == 1)
        e = launch_kernel(attend_tc_kernel<true>, dim3(grid), dim3(tc::THREADS), tc::SMEM_K1, st, pdl,
                          q, k, v, index, lce_w, lce_b, o, lse, status, d, tiles);
    else
        e = launch_kernel(attend_tc_kernel<false>, dim3(grid), dim3(tc::THREADS), tc::SMEM_KN, st, pdl,
                          q, k, v, index, lce_w, lce_b, o, lse, status, d, tiles);
    count_launch();
    return e;
}

}  // namespace bra

#ifdef BRA_TRACE
extern "C" int bra_debug_read_trace(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, bra::g_trace, sizeof(bra::g_trace));
}
#endif
