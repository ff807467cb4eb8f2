// Routed token-to-token attention + LCE on the 5th-generation tensor cores
// (Eq. 6, Eq. 7 with Eq. 1) as a persistent, warp-specialised pipeline.
//
// Shape handled here: head dim 32, regions of 8 x 8 = 64 tokens, heads in pairs.
// A tile is (image b, query region i, head pair hp) = 64 tokens x 64 channels of O.
// The two heads are stacked into one 128-row MMA tile:
//     rows   0..63  = head A queries, rows 64..127 = head B queries
//     keys   0..63  = head A's routed region, keys 64..127 = head B's
// S = Q K^T is 128 x 128 of which each row uses its own head's 64 columns; P has
// zeros in the off-diagonal blocks, so O = P [V_A; V_B] is exact for both heads.
//
// One CTA per SM walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...  Its warps:
//   warp 0      MMA issuer: tcgen05.mma S = Q K^T (operands in shared memory), then
//               O = P V and l = P 1 with P read from tensor memory; polls the groups
//   warp 1      index feeder: routing index rows -> shared-memory ring, range check
//   warps 2-3   loaders: 16-byte cp.async copies of the Q tile, of the K and V tiles of
//               each routed region (K^g / V^g are never formed in HBM: the routing
//               index only picks the source addresses) and of the V halo, written in
//               the swizzled layouts the MMA descriptors expect.  Many small copies
//               in flight per SM reach a multiple of the bandwidth that one bulk
//               tensor copy per 4-18 KB box does at these box sizes.
//   warps 4..   G consumer groups of 4 warps; group g owns tiles g, g + G, ... and
//               128 TMEM columns: S (fp32) is overwritten in place by P (bf16 pairs,
//               columns 0..63), O lands in columns 64..95 and the row sum in column 96.
//               Per tile: softmax (thread = row), normalised O^att to a staging tile,
//               then LCE (warp = 2 columns of the region, lane = channel pair): 5x5
//               depthwise correlation of V from the halo tile with the weights in
//               registers, + O^att, one bf16 store of O.
// Hand-offs are mbarriers; every wait is bounded and abortable.  Hot loops are kept
// rolled and short: the roles run different code on each scheduler, and straight-line
// per-tile code is bound by instruction fetch.
#include "bra_internal.h"
#include "sm100_ptx.cuh"

namespace bra {

using namespace ptx;

namespace tc {
constexpr int RS = 8;            // region side in tokens
constexpr int HALO = RS + 4;     // 12: region plus the 2-token LCE border
constexpr int G = 3;             // consumer groups
constexpr int THREADS = 128 + G * 128;
constexpr int NQ = 3;            // ring depth: Q tiles
constexpr int NH = 5;            // ring depth: V halo tiles
constexpr int NKV = 3;           // ring depth: K and V tiles of one routed step
constexpr int NIDX = 4;          // ring depth: index rows
constexpr int KCAP = 64;         // largest topk
constexpr int TMEM_COLS = 512;
constexpr int TM_GROUP = 128;    // columns per group: S [0,128) / P [0,64) + O [64,96) + l [96,112)
constexpr int TM_O = 64, TM_L = 96;

constexpr int HALO_BYTES = HALO * HALO * 128;            // 18432
// shared memory map (bytes, from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                                 // NQ  x [128 rows][64 B]  64B swizzle, K-major
constexpr int OFF_K = OFF_Q + NQ * 8192;                 // NKV x [128 keys][64 B]  64B swizzle, K-major
constexpr int OFF_V = OFF_K + NKV * 8192;                // NKV x [128 keys][64 B]  64B swizzle, MN-major
constexpr int OFF_HALO = OFF_V + NKV * 8192;             // NH  x [12][12][64 ch] bf16, linear
constexpr int OFF_ST = OFF_HALO + NH * HALO_BYTES;       // G x [64 tokens][64 ch] fp32, 16B units xor-swizzled
constexpr int OFF_ONES = OFF_ST + G * 16384;             // 1024 B of bf16 1.0 (B operand of the row-sum MMA)
constexpr int OFF_IDX = OFF_ONES + 1024;                 // NIDX x [2 heads][KCAP] int32
constexpr int OFF_BAR = OFF_IDX + NIDX * 2 * KCAP * 4;
// barrier slots
constexpr int B_Q_FULL = 0, B_Q_EMPTY = B_Q_FULL + NQ;
constexpr int B_H_FULL = B_Q_EMPTY + NQ, B_H_EMPTY = B_H_FULL + NH;
constexpr int B_KV_FULL = B_H_EMPTY + NH, B_KV_EMPTY = B_KV_FULL + NKV;
constexpr int B_IDX_FULL = B_KV_EMPTY + NKV, B_IDX_EMPTY = B_IDX_FULL + NIDX;
constexpr int B_S_FULL = B_IDX_EMPTY + NIDX;             // per group: S = Q K^T landed in TMEM
constexpr int B_P_FULL = B_S_FULL + G;                   // per group: P written to TMEM
constexpr int B_O_FULL = B_P_FULL + G;                   // per group: O and l landed in TMEM
constexpr int B_S_EMPTY = B_O_FULL + G;                  // per group: O read, the columns may take the next S
constexpr int B_ST_FULL = B_S_EMPTY + G;                 // per group: O^att staged by all four warps
constexpr int B_ST_EMPTY = B_ST_FULL + G;                // per group: staging tile read by all four warps
constexpr int NBARS = B_ST_EMPTY + G;
constexpr int OFF_MISC = OFF_BAR + NBARS * 8;            // tmem slot, abort flag
constexpr int SMEM_BYTES = OFF_MISC + 16;
constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;            // slack for the manual 1024-byte alignment
static_assert(OFF_K % 1024 == 0 && OFF_V % 1024 == 0 && OFF_HALO % 1024 == 0, "swizzled tiles need 1024-byte alignment");
static_assert(SMEM_ALLOC <= 227 * 1024, "shared memory budget");
static_assert(G * TM_GROUP <= TMEM_COLS && G >= 1 && NH > G, "tensor memory / halo ring budget");
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

struct TileCoord { int b, i, hp, y0, x0, c0; };
__device__ __forceinline__ TileCoord tile_coord(int T, const Dims& dm) {
    TileCoord t;
    const int pairs = dm.heads >> 1;
    t.hp = T % pairs;
    t.i = (T / pairs) % dm.R;
    t.b = T / (pairs * dm.R);
    t.y0 = (t.i / dm.S) * tc::RS;
    t.x0 = (t.i % dm.S) * tc::RS;
    t.c0 = t.hp * 64;
    return t;
}

// The loaders keep up to four cp.async groups in flight; a group's "full" barrier is
// signalled (after a proxy fence: the tiles are read by the tensor core's async proxy)
// once the group has landed.
struct LoadQueue {
    uint64_t* p0 = nullptr;   // youngest
    uint64_t* p1 = nullptr;
    uint64_t* p2 = nullptr;   // oldest
    int lane = 0;
    __device__ __forceinline__ void signal(uint64_t* bar) {
        if (!bar) return;
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar);
    }
    // the copies issued since the last push form a new group whose barrier is `bar`
    __device__ __forceinline__ void push(uint64_t* bar) {
        cp_async_commit();
        cp_async_wait<3>();           // all but the three youngest groups have landed
        signal(p2);
        p2 = p1; p1 = p0; p0 = bar;
    }
    __device__ __forceinline__ void flush() {
        cp_async_wait<0>();
        signal(p2); signal(p1); signal(p0);
        p0 = p1 = p2 = nullptr;
    }
};

// K1: topk == 1 (one routed step per tile: no running maximum, no rescaling of O).
template <bool K1>
__global__ void __launch_bounds__(tc::THREADS, 1)
attend_tc_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                 const __nv_bfloat16* __restrict__ Vg, const int32_t* __restrict__ index,
                 const float* __restrict__ lce_w, const float* __restrict__ lce_b,
                 __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
                 int32_t* __restrict__ status, Dims dm, int num_tiles) {
    using namespace tc;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_MISC + 4);
    int32_t* idx_ring = reinterpret_cast<int32_t*>(smem + OFF_IDX);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int k = K1 ? 1 : dm.topk;
    const int my_tiles = (num_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    // ---- one-time set-up -----------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < NQ; ++s) { mbar_init(bars + B_Q_FULL + s, 2); mbar_init(bars + B_Q_EMPTY + s, 1); }
        for (int s = 0; s < NH; ++s) { mbar_init(bars + B_H_FULL + s, 2); mbar_init(bars + B_H_EMPTY + s, 4); }
        for (int s = 0; s < NKV; ++s) { mbar_init(bars + B_KV_FULL + s, 2); mbar_init(bars + B_KV_EMPTY + s, 1); }
        for (int s = 0; s < NIDX; ++s) { mbar_init(bars + B_IDX_FULL + s, 1); mbar_init(bars + B_IDX_EMPTY + s, 6); }
        for (int g = 0; g < G; ++g) {
            mbar_init(bars + B_S_FULL + g, 1); mbar_init(bars + B_P_FULL + g, 4);
            mbar_init(bars + B_O_FULL + g, 1); mbar_init(bars + B_S_EMPTY + g, 4);
            mbar_init(bars + B_ST_FULL + g, 4); mbar_init(bars + B_ST_EMPTY + g, 4);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, TMEM_COLS);
    if (tid >= 64 && tid < 128)
        *reinterpret_cast<uint4*>(smem + OFF_ONES + (tid - 64) * 16) =
            make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // =========================== MMA issuer =======================================
        // One thread serves all groups: it polls (without blocking) what each group needs
        // next - S for its next routed step once Q, K/V have landed and the group's columns
        // are free, or O = P V once the group has written P - and issues whatever is ready.
        if (lane == 0) {
            constexpr uint32_t IDESC_S = umma_idesc_bf16(128, 128, false, false);
            constexpr uint32_t IDESC_O = umma_idesc_bf16(128, 32, false, true);
            constexpr uint32_t IDESC_L = umma_idesc_bf16(128, 16, false, false);
            const uint64_t ones_desc = umma_smem_desc(smem_u32(smem + OFF_ONES), 128, 256, 0);
            int gn[G], gm[G], gc[G], gphase[G];      // tile, step, units done, 0: S next / 1: PV next
            int live = 0;
#pragma unroll
            for (int g = 0; g < G; ++g) { gn[g] = g; gm[g] = 0; gc[g] = 0; gphase[g] = 0; live += (g < my_tiles); }
            uint32_t idle = 0;
            while (live > 0) {
                bool progress = false;
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    if (gn[g] >= my_tiles) continue;
                    const int n = gn[g], m = gm[g], c = gc[g];
                    const int uid = n * k + m, kv = uid % NKV;
                    const uint32_t tg = tmem + g * TM_GROUP;
                    if (gphase[g] == 0) {
                        const int qs = n % NQ;
                        if (m == 0 && !mbar_test_wait(bars + B_Q_FULL + qs, (n / NQ) & 1)) continue;
                        if (!mbar_test_wait(bars + B_KV_FULL + kv, (uid / NKV) & 1)) continue;
                        if (c > 0 && !mbar_test_wait(bars + B_S_EMPTY + g, (c - 1) & 1)) continue;
                        tc_fence_after_sync();
                        const uint32_t qa = smem_u32(smem + OFF_Q + qs * 8192);
                        const uint32_t ka = smem_u32(smem + OFF_K + kv * 8192);
#pragma unroll
                        for (int ks = 0; ks < 2; ++ks)     // d = 32 = 2 k-steps of 16
                            umma_ss(tg, umma_smem_desc(qa + ks * 32, 16, 512, 4),
                                    umma_smem_desc(ka + ks * 32, 16, 512, 4), IDESC_S, ks);
                        umma_commit(bars + B_S_FULL + g);
                        if (m == k - 1) umma_commit(bars + B_Q_EMPTY + qs);   // Q tile no longer needed
                        gphase[g] = 1;
                        progress = true;
                    } else {
                        if (!mbar_test_wait(bars + B_P_FULL + g, c & 1)) continue;
                        tc_fence_after_sync();
                        const uint64_t vd = umma_smem_desc(smem_u32(smem + OFF_V + kv * 8192), 16, 512, 4);
#pragma unroll 1
                        for (int ks = 0; ks < 8; ++ks) {   // 128 keys = 8 k-steps of 16
                            umma_ts(tg + TM_O, tg + ks * 8, vd + (uint64_t)(ks * 64), IDESC_O, ks);
                            umma_ts(tg + TM_L, tg + ks * 8, ones_desc, IDESC_L, ks);
                        }
                        umma_commit(bars + B_O_FULL + g);
                        umma_commit(bars + B_KV_EMPTY + kv);
                        gc[g] = c + 1;
                        gphase[g] = 0;
                        if (m + 1 == k) { gm[g] = 0; gn[g] = n + G; if (n + G >= my_tiles) --live; }
                        else gm[g] = m + 1;
                        progress = true;
                    }
                }
                if (progress) { idle = 0; continue; }
                if (++idle > POLL_LIMIT) { *abort_flag = 1; break; }
                if ((idle & 63u) == 0 && *abort_flag) break;
            }
        }
    } else if (warp == 1) {
        // =========================== index feeder =====================================
        for (int n = 0; n < my_tiles; ++n) {
            const TileCoord t = tile_coord(blockIdx.x + n * gridDim.x, dm);
            const int slot = n % NIDX;
            // entries of both heads' rows: lane-parallel global loads issued before the wait
            const int hA = 2 * t.hp, hB = hA + 1;
            const int hiA = dm.heads_i == 1 ? 0 : hA, hiB = dm.heads_i == 1 ? 0 : hB;
            const int32_t* rowA = index + (((size_t)t.b * dm.heads_i + hiA) * dm.R + t.i) * k;
            const int32_t* rowB = index + (((size_t)t.b * dm.heads_i + hiB) * dm.R + t.i) * k;
            int32_t vals[(2 * KCAP + 31) / 32];
#pragma unroll
            for (int e = 0; e < (2 * KCAP + 31) / 32; ++e) {
                const int id = e * 32 + lane;
                vals[e] = 0;
                if (id < 2 * k) {
                    int r = id < k ? __ldg(rowA + id) : __ldg(rowB + id - k);
                    if (r < 0 || r >= dm.R) { record_error(status, BRA_ERR_INDEX, r); r = -1; }
                    vals[e] = r;
                }
            }
            if (!mbar_wait_abortable(bars + B_IDX_EMPTY + slot, ((n / NIDX) & 1) ^ 1, abort_flag)) break;
            int32_t* rows = idx_ring + slot * 2 * KCAP;
#pragma unroll
            for (int e = 0; e < (2 * KCAP + 31) / 32; ++e) {
                const int id = e * 32 + lane;
                if (id < 2 * k) rows[id < k ? id : KCAP + id - k] = vals[e];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + B_IDX_FULL + slot);
        }
    } else if (warp < 4) {
        // =========================== loaders ==========================================
        // Thread lt copies 16-byte chunk c = lt & 7 of the 128-byte channel row (both heads)
        // of token column tx = lt >> 3 in each of the 8 token rows of a region: a warp covers
        // 512 contiguous bytes per instruction.  Chunks 0-3 are head A, 4-7 head B; inside
        // a head's [token][64 B] tile the chunk index is xor-ed with (token >> 1) & 3, the
        // 64-byte swizzle that the MMA descriptors name.
        const int lt = tid - 64;
        const int c = lt & 7, tx = lt >> 3;
        const int head = c >> 2;
        const uint32_t tile_off = head * 4096 + tx * 64 + (((c & 3) ^ ((tx >> 1) & 3)) << 4);
        const size_t row_bytes = (size_t)dm.W * dm.C * 2;
        const uint32_t q_dst = smem_u32(smem + OFF_Q) + tile_off;
        const uint32_t k_dst = smem_u32(smem + OFF_K) + tile_off;
        const uint32_t v_dst = smem_u32(smem + OFF_V) + tile_off;
        const uint32_t h_dst = smem_u32(smem + OFF_HALO) + tx * 128 + c * 16;
        const uint8_t* Qb = reinterpret_cast<const uint8_t*>(Qg);
        const uint8_t* Kb = reinterpret_cast<const uint8_t*>(Kg);
        const uint8_t* Vb = reinterpret_cast<const uint8_t*>(Vg);
        LoadQueue lq;
        lq.lane = lane;
        bool ok = true;
        int u = 0;
        auto wait_for = [&](uint64_t* bar, uint32_t parity) -> bool {
            if (mbar_test_wait(bar, parity)) return true;
            lq.flush();       // never sit on landed tiles while waiting
            return mbar_wait_abortable(bar, parity, abort_flag);
        };
        for (int n = 0; n < my_tiles && ok; ++n) {
            const TileCoord t = tile_coord(blockIdx.x + n * gridDim.x, dm);
            const size_t img = (size_t)t.b * dm.H * row_bytes;
            const size_t in_row = (size_t)t.c0 * 2 + c * 16;           // byte offset inside a token's channels
            {   // ---- Q tile ----
                const int s = n % NQ;
                if (!(ok = wait_for(bars + B_Q_EMPTY + s, ((n / NQ) & 1) ^ 1))) break;
                const uint8_t* src = Qb + img + (size_t)t.y0 * row_bytes + (size_t)(t.x0 + tx) * dm.C * 2 + in_row;
                const uint32_t dst = q_dst + s * 8192;
#pragma unroll
                for (int i = 0; i < 8; ++i) cp_async_16(dst + i * 512, src + i * row_bytes, 16);
                lq.push(bars + B_Q_FULL + s);
            }
            const int slot = n % NIDX;
            if (!(ok = wait_for(bars + B_IDX_FULL + slot, (n / NIDX) & 1))) break;
            const int32_t* rows = idx_ring + slot * 2 * KCAP + head * KCAP;
            for (int m = 0; m < k; ++m, ++u) {
                // ---- K and V tiles of routed step m: this thread's head picks the region ----
                const int kv = u % NKV;
                if (!(ok = wait_for(bars + B_KV_EMPTY + kv, ((u / NKV) & 1) ^ 1))) break;
                int r = rows[m];
                r = r < 0 ? 0 : r;              // an invalid entry loads region 0; its P is zero
                const size_t off = img + (size_t)((r / dm.S) * RS) * row_bytes +
                                   (size_t)((r % dm.S) * RS + tx) * dm.C * 2 + in_row;
                const uint32_t kd = k_dst + kv * 8192, vd = v_dst + kv * 8192;
#pragma unroll
                for (int i = 0; i < 8; ++i) cp_async_16(kd + i * 512, Kb + off + i * row_bytes, 16);
#pragma unroll
                for (int i = 0; i < 8; ++i) cp_async_16(vd + i * 512, Vb + off + i * row_bytes, 16);
                lq.push(bars + B_KV_FULL + kv);
            }
            if (!ok) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + B_IDX_EMPTY + slot);
            if (dm.lce) {
                // ---- V halo: 12 x 12 tokens x 128 B around the region, zeros outside the map ----
                const int hs = n % NH;
                if (!(ok = wait_for(bars + B_H_EMPTY + hs, ((n / NH) & 1) ^ 1))) break;
                const uint32_t dst = h_dst + hs * HALO_BYTES;
                int hy = 0, hx = tx;
#pragma unroll 1
                for (int i = 0; i < 18; ++i) {
                    const int y = t.y0 - 2 + hy, x = t.x0 - 2 + hx;
                    const bool inb = (unsigned)y < (unsigned)dm.H && (unsigned)x < (unsigned)dm.W;
                    const uint8_t* src = inb ? Vb + img + (size_t)y * row_bytes + (size_t)x * dm.C * 2 + in_row : Vb;
                    cp_async_16(dst + i * 1024, src, inb ? 16u : 0u);
                    hx += 8;
                    if (hx >= HALO) { hx -= HALO; ++hy; }
                }
                lq.push(bars + B_H_FULL + hs);
            }
        }
        lq.flush();           // also on the way out after an abort: nothing stays in flight
    } else {
        // =========================== consumer groups ==================================
        const int g = (warp - 4) >> 2;                 // group
        const int wq = warp & 3;                       // TMEM lane quadrant of this warp
        const int row = wq * 32 + lane;                // row of the stacked tile = TMEM lane
        const int head_half = row >> 6;                // 0: head A, 1: head B
        const int tq = row & 63;                       // query token inside the region
        const uint32_t tg = tmem + ((uint32_t)(wq * 32) << 16) + g * TM_GROUP;
        const uint32_t s_addr = tg + head_half * 64;   // this row's 64 scores
        const uint32_t p_addr = tg + head_half * 32;   // this row's 64 probabilities (bf16 pairs)
        const uint32_t z_addr = tg + (head_half ^ 1) * 32;   // the other head's keys: zeros
        const float sl2 = dm.scale * 1.4426950408889634f;
        const int xl0 = 2 * wq;                        // LCE: this warp's two columns of the region
        uint8_t* const stage = smem + OFF_ST + g * 16384;
        float2 wv[25];
#pragma unroll
        for (int q = 0; q < 25; ++q) wv[q] = make_float2(0.f, 0.f);
        float2 bias2 = make_float2(0.f, 0.f);
        int hp_loaded = -1;
        int c = 0;                                     // routed steps done by this group
        int j = 0;                                     // tiles done by this group
        bool ok = true;
        for (int n = g; n < my_tiles && ok; n += G, ++j) {
            const TileCoord t = tile_coord(blockIdx.x + n * gridDim.x, dm);
            const int slot = n % NIDX;
            if (dm.lce && t.hp != hp_loaded) {
                const float* wp = lce_w + (size_t)(t.c0 + 2 * lane) * 25;
#pragma unroll
                for (int q = 0; q < 25; ++q) wv[q] = make_float2(__ldg(wp + q), __ldg(wp + 25 + q));
                if (lce_b) bias2 = make_float2(__ldg(lce_b + t.c0 + 2 * lane), __ldg(lce_b + t.c0 + 2 * lane + 1));
                hp_loaded = t.hp;
            }
            if (!(ok = mbar_wait_abortable(bars + B_IDX_FULL + slot, (n / NIDX) & 1, abort_flag))) break;
            const int32_t* rows = idx_ring + slot * 2 * KCAP + head_half * KCAP;

            // ---- softmax over the routed steps (thread = row) ----
            float m_run = -INFINITY, l_run = 0.f;
            float o_acc[32];
#pragma unroll
            for (int q = 0; q < 32; ++q) o_acc[q] = 0.f;
            for (int m = 0; m < k; ++m, ++c) {
                const bool valid = rows[m] >= 0;
                if (!(ok = mbar_wait_abortable(bars + B_S_FULL + g, c & 1, abort_flag))) break;
                tc_fence_after_sync();
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
                // pass 2: P = exp2(S * scale * log2 e - max), bf16 pairs written over the
                // columns of S already consumed (column j of P never outruns column 2j of S)
                const float2 sl2v = make_float2(sl2, sl2), mnegv = make_float2(mneg, mneg);
#pragma unroll 1
                for (int cc = 0; cc < 64; cc += 16) {
                    uint32_t r[16], pk[8];
                    tmem_ld_32x32b_x16(s_addr + cc, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 16; q += 2) {
                        const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[q]), __uint_as_float(r[q + 1])), sl2v, mnegv);
                        pk[q >> 1] = valid ? pack_bf16(ex2f(a.x), ex2f(a.y)) : 0u;
                    }
                    tmem_st_32x32b_x8(p_addr + (cc >> 1), pk);
                }
                {
                    uint32_t z[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) z[q] = 0u;
#pragma unroll
                    for (int cc = 0; cc < 32; cc += 8) tmem_st_32x32b_x8(z_addr + cc, z);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + B_P_FULL + g);
                // ---- O and the row sum of this step ----
                if (!(ok = mbar_wait_abortable(bars + B_O_FULL + g, c & 1, abort_flag))) break;
                tc_fence_after_sync();
                uint32_t oraw[32], lraw[1];
                tmem_ld_32x32b_x32(tg + TM_O, oraw);
                tmem_ld_32x32b_x1(tg + TM_L, lraw);
                tmem_ld_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + B_S_EMPTY + g);
                if (K1) {
                    l_run = __uint_as_float(lraw[0]);
#pragma unroll
                    for (int q = 0; q < 32; ++q) o_acc[q] = __uint_as_float(oraw[q]);
                } else {
                    l_run = fmaf(l_run, corr, __uint_as_float(lraw[0]));
#pragma unroll
                    for (int q = 0; q < 32; ++q) o_acc[q] = fmaf(o_acc[q], corr, __uint_as_float(oraw[q]));
                }
            }
            if (!ok) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + B_IDX_EMPTY + slot);

            // ---- normalise, stage O^att as fp32 [64 tokens][64 ch] for the LCE mapping ----
            {
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
                uint8_t* srow = stage + tq * 256;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int chunk = head_half * 8 + q;
                    *reinterpret_cast<float4*>(srow + ((chunk ^ (tq & 7)) << 4)) =
                        make_float4(o_acc[4 * q] * inv, o_acc[4 * q + 1] * inv, o_acc[4 * q + 2] * inv, o_acc[4 * q + 3] * inv);
                }
                if (lse)
                    lse[((size_t)t.b * dm.heads + 2 * t.hp + head_half) * dm.N + (size_t)(t.y0 + tq / RS) * dm.W + t.x0 + tq % RS] =
                        (m_run + log2f(l_run)) * 0.6931471805599453f;
            }
            // group-wide hand-over of the staging tile (an mbarrier, so that the wait can give up)
            __syncwarp();
            if (lane == 0) mbar_arrive(bars + B_ST_FULL + g);
            if (!(ok = mbar_wait_abortable(bars + B_ST_FULL + g, j & 1, abort_flag))) break;

            // ---- LCE + store (warp = 2 columns, lane = channel pair) ----
            // One rolled loop over the 12 input rows of the halo: row yy feeds output rows
            // yy - ti through tap row ti, so running sums slide down the region; the sum that
            // took tap row 4 is complete and leaves as O = O^att + LCE(V).
            const int hs = n % NH;
            if (dm.lce && !(ok = mbar_wait_abortable(bars + B_H_FULL + hs, (n / NH) & 1, abort_flag))) break;
            const uint32_t* halo = reinterpret_cast<const uint32_t*>(smem + OFF_HALO + hs * HALO_BYTES) + lane;
            uint32_t* out = reinterpret_cast<uint32_t*>(O) +
                            ((((size_t)t.b * dm.H + t.y0) * dm.W + t.x0 + xl0) * dm.C + t.c0) / 2 + lane;
            float2 p1[2], p2[2], p3[2], p4[2];
#pragma unroll
            for (int xx = 0; xx < 2; ++xx) { p1[xx] = bias2; p2[xx] = bias2; p3[xx] = bias2; p4[xx] = bias2; }
#pragma unroll 1
            for (int yy = dm.lce ? 0 : 4; yy < HALO; ++yy) {
                float2 e[2];
#pragma unroll
                for (int xx = 0; xx < 2; ++xx) e[xx] = p4[xx];
                if (dm.lce) {
                    float2 v[6];
#pragma unroll
                    for (int xx = 0; xx < 6; ++xx) {
                        const uint32_t w = halo[(yy * HALO + xl0 + xx) * 32];
                        v[xx] = make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
                    }
                    // output row y = yy - ti takes tap row ti of this input row; rows outside
                    // the region are skipped (their sums are never read)
                    if (yy >= 4) {
#pragma unroll
                        for (int xx = 0; xx < 2; ++xx)
#pragma unroll
                            for (int tj = 0; tj < 5; ++tj) e[xx] = __ffma2_rn(wv[20 + tj], v[xx + tj], e[xx]);
                    }
                    if (yy >= 3 && yy < 11) {
#pragma unroll
                        for (int xx = 0; xx < 2; ++xx) {
                            p4[xx] = p3[xx];
#pragma unroll
                            for (int tj = 0; tj < 5; ++tj) p4[xx] = __ffma2_rn(wv[15 + tj], v[xx + tj], p4[xx]);
                        }
                    }
                    if (yy >= 2 && yy < 10) {
#pragma unroll
                        for (int xx = 0; xx < 2; ++xx) {
                            p3[xx] = p2[xx];
#pragma unroll
                            for (int tj = 0; tj < 5; ++tj) p3[xx] = __ffma2_rn(wv[10 + tj], v[xx + tj], p3[xx]);
                        }
                    }
                    if (yy >= 1 && yy < 9) {
#pragma unroll
                        for (int xx = 0; xx < 2; ++xx) {
                            p2[xx] = p1[xx];
#pragma unroll
                            for (int tj = 0; tj < 5; ++tj) p2[xx] = __ffma2_rn(wv[5 + tj], v[xx + tj], p2[xx]);
                        }
                    }
                    if (yy < 8) {
#pragma unroll
                        for (int xx = 0; xx < 2; ++xx) {
                            p1[xx] = bias2;
#pragma unroll
                            for (int tj = 0; tj < 5; ++tj) p1[xx] = __ffma2_rn(wv[tj], v[xx + tj], p1[xx]);
                        }
                    }
                }
                if (yy >= 4) {
                    const int y = yy - 4;
#pragma unroll
                    for (int xx = 0; xx < 2; ++xx) {
                        const int tk = y * RS + xl0 + xx;
                        const float2 att = *reinterpret_cast<const float2*>(
                            stage + tk * 256 + (((lane >> 1) ^ (tk & 7)) << 4) + (lane & 1) * 8);
                        out[((size_t)y * dm.W + xx) * (dm.C / 2)] = pack_bf16(att.x + e[xx].x, att.y + e[xx].y);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                if (dm.lce) mbar_arrive(bars + B_H_EMPTY + hs);
                mbar_arrive(bars + B_ST_EMPTY + g);
            }
            // the staging tile may be overwritten once all four warps have read it
            if (!(ok = mbar_wait_abortable(bars + B_ST_EMPTY + g, j & 1, abort_flag))) break;
        }
    }

    // ---- teardown ------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && *abort_flag) record_error(status, BRA_ERR_TIMEOUT, blockIdx.x);
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
           d.topk <= tc::KCAP && (long long)d.B * d.R * (d.heads / 2) < (1ll << 30);
}

cudaError_t launch_attend_tc(const Dims& d, const void* Q, const void* K, const void* V,
                             const int32_t* index, const float* lce_w, const float* lce_b,
                             void* O, float* lse, int32_t* status, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_ALLOC);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(attend_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_ALLOC);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const int tiles = d.B * d.R * (d.heads / 2);
    const int sms = sm_count();
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(Q);
    const __nv_bfloat16* k = static_cast<const __nv_bfloat16*>(K);
    const __nv_bfloat16* v = static_cast<const __nv_bfloat16*>(V);
    if (d.topk == 1)
        attend_tc_kernel<true><<<grid, tc::THREADS, tc::SMEM_ALLOC, st>>>(
            q, k, v, index, lce_w, lce_b, static_cast<__nv_bfloat16*>(O), lse, status, d, tiles);
    else
        attend_tc_kernel<false><<<grid, tc::THREADS, tc::SMEM_ALLOC, st>>>(
            q, k, v, index, lce_w, lce_b, static_cast<__nv_bfloat16*>(O), lse, status, d, tiles);
    count_launch();
    return cudaGetLastError();
}

}  // namespace bra
