// Routed token-to-token attention + LCE on the 5th-generation tensor cores for topk = 1
// (Eq. 6, Eq. 7 with Eq. 1): every query region attends to one routed region per head, so a tile
// needs one S = Q K^T, one softmax without running maximum, and one O = P V.
//
// Tile layout, thread mappings and shared-memory map are those of attend_tc.cu (two heads stacked
// into a 128-row MMA tile, 128-thread CTAs, four per SM).  What differs is the schedule: the tensor
// core works one tile ahead of the threads.  While the threads run the softmax and P V of tile n,
// Q and K of tile n + 1 stream into the buffers S_n has just released; S_{n+1} = Q K^T is issued
// before the LCE of tile n starts and completes underneath it, so a tile never waits for its first
// MMA.  V of tile n + 1 follows once the staging tile that overlays it has been read, the halo
// once the LCE is done.  Per tile:
//   wait S_n (issued during tile n - 1)  ->  copies of Q, K of tile n + 1 go out
//   softmax, P to TMEM  ->  O = P V  ->  normalised O^att to the fp32 staging tile
//   S_{n+1} issued  ->  LCE sums start from O^att  ->  copy of V of tile n + 1 goes out
//   LCE (5x5 depthwise correlation of V from the halo tile), one bf16 store of O
//   ->  copy of the halo of tile n + 1 goes out
// Every wait on an MMA is bounded.
#include "attend_tc_common.cuh"

namespace bra {

__global__ void __launch_bounds__(tc::THREADS, 4)
attend_tc_k1_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
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
    const int inv_s = (1 << 20) / dm.S + 1;            // i / S == (i * inv_s) >> 20 for i < 4096
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
    const size_t img_bytes = (size_t)dm.H * row_bytes;
    const size_t thr_off = (size_t)lrow * row_bytes + (size_t)tx * dm.C * 2 + c * 16;   // this thread's chunk inside a region
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

    auto coord_of = [&](int b, int i, int hp) -> TileCoord {
        TileCoord t;
        t.b = b; t.i = i; t.hp = hp;
        const int ry = (i * inv_s) >> 20;
        t.y0 = ry * RS;
        t.x0 = (i - ry * dm.S) * RS;
        t.c0 = hp * 64;
        return t;
    };
    // byte offset of this thread's chunk of region r (image b, head pair's 64 channels at c0)
    auto region_off = [&](int b, int r, int c0) -> size_t {
        const int ry = (r * inv_s) >> 20, rx = r - ry * dm.S;
        return (size_t)b * img_bytes + (size_t)(ry * RS) * row_bytes + (size_t)(rx * RS) * dm.C * 2 + (size_t)c0 * 2 + thr_off;
    };
    // routing entries (head A, head B) of a unit = (tile, routed step); -1: out of range.  The index may
    // come from a kernel this one overlaps (programmatic dependent launch): coherent loads after
    // pdl_wait(), never the read-only path, whose loads the compiler may move above the wait
    auto read_entries = [&](const TileCoord& t, int m) -> int2 {
        const int hA = 2 * t.hp, hB = hA + 1;
        const int hiA = dm.heads_i == 1 ? 0 : hA, hiB = dm.heads_i == 1 ? 0 : hB;
        int ra = __ldcg(index + (((size_t)t.b * dm.heads_i + hiA) * dm.R + t.i) * dm.topk + m);
        int rb = __ldcg(index + (((size_t)t.b * dm.heads_i + hiB) * dm.R + t.i) * dm.topk + m);
        if (ra < 0 || ra >= dm.R) { record_error(status, BRA_ERR_INDEX, ra); ra = -1; }
        if (rb < 0 || rb >= dm.R) { record_error(status, BRA_ERR_INDEX, rb); rb = -1; }
        return make_int2(ra, rb);
    };
    auto load_k = [&](const TileCoord& t, int2 ent, int buf) {
        int r = lhead ? ent.y : ent.x;
        r = r < 0 ? 0 : r;                  // an invalid entry loads region 0; its P is zero
        const uint8_t* src = Kb + region_off(t.b, r, t.c0);
        const uint32_t kd = sm_base + (buf ? OFF_KV1 : OFF_K) + tile_off;
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async_16(kd + i * 512, src + i * row_bytes, 16);
    };
    auto load_v = [&](const TileCoord& t, int2 ent, int buf) {
        int r = lhead ? ent.y : ent.x;
        r = r < 0 ? 0 : r;
        const uint8_t* src = Vb + region_off(t.b, r, t.c0);
        const uint32_t vd = sm_base + (buf ? OFF_KV1 + 8192 : OFF_V) + v_off;
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async_16(vd + i * 1024, src + i * row_bytes, 16);
    };
    auto load_q = [&](const TileCoord& t) {
        const uint8_t* src = Qb + region_off(t.b, t.i, t.c0);
        const uint32_t dst = sm_base + OFF_Q + tile_off;
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async_16(dst + i * 512, src + i * row_bytes, 16);
    };
    // halo: thread (column hx = tid >> 3 of the 12, 16-byte chunk c) copies its chunk of every one of the
    // 12 halo rows; threads 96..127 have no column.  Zeros outside the map (the conv's zero padding).
    const int hx = tid >> 3;
    auto load_halo = [&](const TileCoord& t) {
        if (!dm.lce || hx >= HALO) return;
        const bool col_in = (t.x0 + hx >= 2) && (t.x0 + hx - 2 < dm.W);
        const uint8_t* src = Vb + (size_t)t.b * img_bytes + (size_t)t.x0 * dm.C * 2 + (size_t)t.c0 * 2 + c * 16 +
                             (ptrdiff_t)(hx - 2) * dm.C * 2;
        const uint32_t hd = sm_base + OFF_HALO + tid * 16;
#pragma unroll
        for (int hy = 0; hy < HALO; ++hy) {
            const int y = t.y0 + hy - 2;
            const bool inb = col_in && y >= 0 && y < dm.H;
            cp_async_16(hd + hy * (HALO * 128), inb ? src + (ptrdiff_t)y * (ptrdiff_t)row_bytes : Vb, inb ? 16u : 0u);
        }
    };

    auto issue_s = [&]() {                  // one thread: S = Q K^T for the tile whose Q and K are in shared memory
        tc_fence_after_sync();
        const uint32_t qa = sm_base + OFF_Q, ka = sm_base + OFF_K;
#pragma unroll
        for (int ks = 0; ks < 2; ++ks)         // d = 32 = 2 k-steps of 16
            umma_ss(tmem, umma_smem_desc(qa + ks * 32, 16, 512, 4),
                    umma_smem_desc(ka + ks * 32, 16, 512, 4), IDESC_S, ks);
        umma_commit(bar_s);
    };

    bool ok = true;
    TileCoord t = coord_of(walk.b, walk.i, walk.hp);
    // copies of a tile go out in three groups: (Q, K), then V, then the halo.
    // Q is an input of the call: its copy (and everything above) overlaps the tail of the kernel before
    // (routing, in a forward call); only the routing index has to wait for it
    if (my_tiles > 0) load_q(t);
    pdl_wait();
    int2 ent = make_int2(0, 0);             // routing entries (head A, head B) of the tile in hand
    if (my_tiles > 0) {
        ent = read_entries(t, 0);
        load_k(t, ent, 0);
    }
    cp_async_commit();
    if (my_tiles > 0) load_v(t, ent, 0);
    cp_async_commit();
    if (my_tiles > 0) load_halo(t);
    cp_async_commit();
    cp_async_wait<2>();
    fence_proxy_async_smem();
    __syncthreads();
    if (tid == 0 && my_tiles > 0) issue_s();

    for (int n = 0; n < my_tiles; ++n) {
        if (dm.lce && t.hp != hp_loaded) {
            const float* wp = lce_w + (size_t)(t.c0 + 2 * lane) * 25;
#pragma unroll
            for (int q = 0; q < 25; ++q) wv[q] = make_float2(__ldg(wp + q), __ldg(wp + 25 + q));
            if (lce_b) bias2 = make_float2(__ldg(lce_b + t.c0 + 2 * lane), __ldg(lce_b + t.c0 + 2 * lane + 1));
            hp_loaded = t.hp;
        }
        const bool has_next = n + 1 < my_tiles;
        if (has_next) walk.next();
        const TileCoord tn = has_next ? coord_of(walk.b, walk.i, walk.hp) : t;
        int2 ent_n = ent;
        if (has_next) ent_n = read_entries(tn, 0);

        // ---- S of this tile is in TMEM (issued a tile ago) ----
        if (warp == 0) ok = mbar_wait(bar_s, n & 1, POLL_LIMIT);     // one warp polls, the rest sleep at the barrier
        if (!__syncthreads_and(ok)) { ok = false; break; }
        tc_fence_after_sync();
        // the MMA has read Q and K: the next tile's take their place
        if (has_next) { load_q(tn); load_k(tn, ent_n, 0); }
        cp_async_commit();

        // ---- softmax: thread = row.  Pass 1: row maximum ----
        const bool valid = (head_half ? ent.y : ent.x) >= 0;
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
        const float mx = fmaxf(m0, m1) * sl2;                          // sl2 > 0
        // an out-of-range routing entry: every probability of the row is exp2(-inf) = 0
        const float mneg = valid ? -mx : -INFINITY;
        // pass 2: P = exp2(S * scale * log2 e - max), bf16 pairs written over the columns
        // of S already consumed (column j of P never outruns column 2j of S); row sum
        const float2 sl2v = make_float2(valid ? sl2 : 0.f, valid ? sl2 : 0.f), mnegv = make_float2(mneg, mneg);
        float2 sum2 = make_float2(0.f, 0.f);
#pragma unroll 1
        for (int cc = 0; cc < 64; cc += 16) {
            uint32_t r[16], pk[8];
            tmem_ld_32x32b_x16(s_addr + cc, r);
            tmem_ld_wait();
#pragma unroll
            for (int q = 0; q < 16; q += 2) {
                const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[q]), __uint_as_float(r[q + 1])), sl2v, mnegv);
                const float2 pe = make_float2(ex2f(a.x), ex2f(a.y));
                sum2 = __fadd2_rn(sum2, pe);
                pk[q >> 1] = pack_bf16(pe.x, pe.y);
            }
            tmem_st_32x32b_x8(p_addr + (cc >> 1), pk);
        }
        tmem_st_wait();
        // V and the halo of this tile have landed (the next tile's Q and K may still be in flight)
        cp_async_wait<1>();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after_sync();
            const uint64_t vd = umma_smem_desc(sm_base + OFF_V, 16, 1024, 2);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)         // 64 keys = 4 k-steps of 16 (2048 B of V each)
                umma_ts(tmem + TM_O, tmem + ks * 8, vd + (uint64_t)(ks * 128), IDESC_O, ks);
            umma_commit(bar_o);
        }
        if (warp == 0) ok = mbar_wait(bar_o, n & 1, POLL_LIMIT);
        if (!__syncthreads_and(ok)) { ok = false; break; }
        tc_fence_after_sync();
        // ---- normalise, stage O^att as fp32 [64 tokens][64 ch] (16-byte units xor-swizzled) ----
        {
            uint32_t oraw[32];
            tmem_ld_32x32b_x32(o_addr, oraw);
            tmem_ld_wait();
            const float l_run = sum2.x + sum2.y;
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            const uint32_t srow = sm_base + OFF_ST + tq * 256;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int chunk = head_half * 8 + q;
                sts_f32x4(srow + ((chunk ^ (tq & 7)) << 4),
                          __uint_as_float(oraw[4 * q]) * inv, __uint_as_float(oraw[4 * q + 1]) * inv,
                          __uint_as_float(oraw[4 * q + 2]) * inv, __uint_as_float(oraw[4 * q + 3]) * inv);
            }
            if (lse)
                lse[((size_t)t.b * dm.heads + 2 * t.hp + head_half) * dm.N + (size_t)(t.y0 + tq / RS) * dm.W + t.x0 + tq % RS] =
                    (valid ? mx + log2f(l_run) : -INFINITY) * 0.6931471805599453f;
        }
        // Q and K of the next tile have landed; TMEM has been read: the tensor core starts on the next tile
        cp_async_wait<0>();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        if (tid == 0 && has_next) issue_s();

        // ---- LCE + store ----
        // Input row yy of the halo feeds output rows yy - ti through tap row ti.  Fully unrolled:
        // the 8 x 2 output sums of this thread's channel pair sit in registers under fixed names,
        // starting from O^att (+ bias).
        {
            const uint32_t halo = sm_base + OFF_HALO + (xl0 * 32 + lane) * 4;
            const uint32_t stage = sm_base + OFF_ST + xl0 * 256 + (lane & 1) * 8;
            // staging token tk = y * 8 + xl0 + xx: its 16-byte unit index is xor-ed with tk & 7
            const uint32_t sw0 = (((lane >> 1) ^ (xl0 & 7)) << 4), sw1 = (((lane >> 1) ^ ((xl0 + 1) & 7)) << 4);
            float2 acc[8][2];
#pragma unroll
            for (int y = 0; y < 8; ++y)
#pragma unroll
                for (int xx = 0; xx < 2; ++xx)
                    acc[y][xx] = __fadd2_rn(lds_f32x2(stage + (y * RS + xx) * 256 + (xx ? sw1 : sw0)), bias2);
            __syncthreads();                // the staging tile has been read: V of the next tile takes its place
            if (has_next) load_v(tn, ent_n, 0);
            cp_async_commit();
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
            uint32_t* out = reinterpret_cast<uint32_t*>(O) +
                            ((((size_t)t.b * dm.H + t.y0) * dm.W + t.x0 + xl0) * dm.C + t.c0) / 2 + lane;
            const size_t out_row = (size_t)dm.W * (dm.C / 2);
#pragma unroll
            for (int y = 0; y < 8; ++y) {
#pragma unroll
                for (int xx = 0; xx < 2; ++xx) out[xx * (dm.C / 2)] = pack_bf16(acc[y][xx].x, acc[y][xx].y);
                out += out_row;
            }
        }
        __syncthreads();                    // the halo is free
        if (has_next) load_halo(tn);
        cp_async_commit();
        t = tn;
        ent = ent_n;
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
cudaError_t launch_attend_tc_k1(const Dims& d, const void* Q, const void* K, const void* V,
                                const int32_t* index, const float* lce_w, const float* lce_b,
                                void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel) {
    static PerDeviceOnce once;
    cudaError_t e = once.run([]() -> cudaError_t {
        cudaError_t a = cudaFuncSetAttribute(attend_tc_k1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_K1);
        if (a != cudaSuccess) return a;
        // several CTAs per SM: ask for the largest shared-memory carve-out
        return cudaFuncSetAttribute(attend_tc_k1_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    });
    if (e != cudaSuccess) return e;
    const int tiles = d.B * d.R * (d.heads / 2);
    const int resident = tc_sm_count() * 4;
    const unsigned grid = (unsigned)(tiles < resident ? tiles : resident);
    e = launch_kernel(attend_tc_k1_kernel, dim3(grid), dim3(tc::THREADS), tc::SMEM_K1, st, after_own_kernel,
                      static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(K),
                      static_cast<const __nv_bfloat16*>(V), index, lce_w, lce_b,
                      static_cast<__nv_bfloat16*>(O), lse, status, d, tiles);
    count_launch();
    return e;
}

}  // namespace bra
