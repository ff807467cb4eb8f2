// Routed token-to-token attention + LCE on the 5th-generation tensor cores for large
// regions (Eq. 6, Eq. 7 with Eq. 1): head dim 32, bf16, regions 16 tokens wide and a
// multiple of 8 tokens high (e.g. 16 x 16 = 256 tokens: 512 x 512 inputs at stride 4
// with S = 8).  This is the tensor-/exp-bound regime: every query meets topk * n_r keys.
//
// A tile is (image b, query region i, head h, block of 8 token rows) = 128 queries of one
// head = the 128 rows of a tcgen05 MMA tile.  The routed keys stream by in blocks of 128
// (8 token rows of a routed region), flash-attention style:
//   all threads   cp.async copies of Q (once per tile), of the K and V blocks (double-
//                 buffered, one block ahead) and of the 12 x 20 V halo, in the 64-byte
//                 swizzled layout of the MMA descriptors.  K^g / V^g are never formed in
//                 HBM: the routing index only picks the source addresses.
//   one thread    tcgen05.mma S = Q K^T (128 x 128, fp32 in TMEM)
//   thread = row  online softmax: running maximum, P (bf16 pairs) written over S in TMEM
//   one thread    tcgen05.mma O_blk = P V with P read from TMEM; rescaled sum kept in registers
//   after the last block: normalised O^att to an fp32 staging tile, then LCE (thread =
//   channel pair x 2 columns x 8 rows, sums in registers) + O^att, one bf16 store of O.
// 128-thread CTAs, four per SM, each walking its own tiles.  Every wait on an MMA is bounded.
#include "bra_internal.h"
#include "sm100_ptx.cuh"

namespace bra {

using namespace ptx;

namespace tw {
constexpr int WS = 16;           // region width in tokens
constexpr int RT = 8;            // token rows per tile: RT * WS = 128 queries
constexpr int HROWS = RT + 4, HCOLS = WS + 4;
constexpr int THREADS = 128;
constexpr int KCAP = 64;         // largest topk
constexpr int TMEM_COLS = 128;   // S [0,128) fp32; then P [0,64) bf16 pairs + O [64,96)
constexpr int TM_O = 64;
constexpr int HALO_BYTES = HROWS * HCOLS * 64;           // 15360
// shared memory map (bytes, from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                                 // [128 rows][64 B]  64B swizzle, K-major
constexpr int OFF_ST = 0;                                // [128 tokens][32 ch] fp32: over Q and K buffer 0 (dead by then)
constexpr int OFF_KV = 8192;                             // 2 x { K [128 keys][64 B], V [128 keys][64 B] }, 64B swizzle
constexpr int OFF_HALO = OFF_KV + 2 * 16384;             // [12][20][32 ch] bf16, linear
constexpr int OFF_BAR = OFF_HALO + HALO_BYTES;
constexpr int ALIGN = 512;                               // the 64-byte swizzle repeats every 512 bytes
constexpr int OFF_ENT = OFF_BAR + 64;                    // the tile's routing entries (KCAP ints)
constexpr int SMEM_BYTES = OFF_ENT + KCAP * 4 + ALIGN;   // + slack for the manual alignment
constexpr uint32_t POLL_LIMIT = 4000000u;
}  // namespace tw

__device__ __forceinline__ float ex2w(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t packw(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

__global__ void __launch_bounds__(tw::THREADS, 4)
attend_tc_wide_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                      const __nv_bfloat16* __restrict__ Vg, const int32_t* index,
                      const float* __restrict__ lce_w, const float* __restrict__ lce_b,
                      __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
                      int32_t* __restrict__ status, Dims dm, int num_tiles) {
    using namespace tw;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + (ALIGN - 1)) & ~uintptr_t(ALIGN - 1));
    uint64_t* bar_s = reinterpret_cast<uint64_t*>(smem + OFF_BAR);       // S landed in TMEM
    uint64_t* bar_o = bar_s + 1;                                         // O landed in TMEM
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_s + 2);
    uint64_t* bar_sh = bar_s + 3;                                        // high half of S landed
    uint32_t* arrivals = reinterpret_cast<uint32_t*>(bar_s + 4);         // threads that have read O out of tensor memory (running count)
    volatile int32_t* ent = reinterpret_cast<volatile int32_t*>(smem + OFF_ENT);
    const uint32_t sm_base = smem_u32(smem);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int RB = dm.hs / RT;                       // row blocks per region
    const int units = dm.topk * RB;                  // key blocks per tile
    const int inv_s = (1 << 20) / dm.S + 1;          // r / S == (r * inv_s) >> 20 for r < 4096

    if (tid == 0) {
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        mbar_init(bar_sh, 1);
        *arrivals = 0;
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    pdl_wait();          // the set-up above may overlap the tail of the kernel before (routing, in bra_forward)

    const size_t tok_bytes = (size_t)dm.C * 2;
    const size_t row_bytes = (size_t)dm.W * tok_bytes;
    // ---- loader mapping: chunk c of token (column tx, rows ly, ly + 2, ly + 4, ly + 6) of an 8 x 16 token block
    const int c = tid & 3, tx = (tid >> 2) & 15, ly = tid >> 6;
    const uint32_t blk_off = (uint32_t)(tid >> 2) * 64 + ((c ^ ((tid >> 3) & 3)) << 4);   // row = tid >> 2, + 32 per step
    auto load_block = [&](uint32_t dst, const uint8_t* base) {   // base: first token of the block, this head's channels
        const uint8_t* src = base + (size_t)ly * row_bytes + (size_t)tx * tok_bytes + c * 16;
#pragma unroll
        for (int i = 0; i < 4; ++i) cp_async_16(dst + blk_off + i * 2048, src + (size_t)(2 * i) * row_bytes, 16);
    };
    // ---- softmax mapping: thread = query row = TMEM lane
    const uint32_t tg = tmem + ((uint32_t)(warp * 32) << 16);
    const float sl2 = dm.scale * 1.4426950408889634f;
    // ---- LCE mapping: channel pair cp, two columns, all 8 rows of the tile
    const int cp = lane & 15;
    const int xl0 = 2 * (warp * 2 + (lane >> 4));

    constexpr uint32_t IDESC_SH = umma_idesc_bf16(128, 64, false, false);
    constexpr uint32_t IDESC_O = umma_idesc_bf16(128, 32, false, true);

    bool ok = true;
    uint32_t n_s = 0, n_o = 0;                       // MMA groups waited for so far on each barrier
    uint32_t n_arr = 0;                              // rounds of `arrivals` so far

    for (int T = blockIdx.x; T < num_tiles && ok; T += gridDim.x) {
        int rem = T;
        const int rb = rem % RB; rem /= RB;
        const int h = rem % dm.heads; rem /= dm.heads;
        const int i = rem % dm.R;
        const int b = rem / dm.R;
        const int y0 = (i / dm.S) * dm.hs + rb * RT, x0 = (i % dm.S) * WS;   // first token of the tile
        const size_t img = (size_t)b * dm.H * row_bytes + (size_t)h * 64;
        const uint8_t* Qb = reinterpret_cast<const uint8_t*>(Qg) + img;
        const uint8_t* Kb = reinterpret_cast<const uint8_t*>(Kg) + img;
        const uint8_t* Vb = reinterpret_cast<const uint8_t*>(Vg) + img;
        const int hi = dm.heads_i == 1 ? 0 : h;
        const int32_t* irow = index + (((size_t)b * dm.heads_i + hi) * dm.R + i) * dm.topk;

        // key block u = (routed slot m, row block of that region); entry -1: out of range, its P is zero
        // (u = m * RB + kb: the launcher keeps R <= 4096, so r / S is a multiply and a shift)
        // the tile's routing entries go to shared memory once (coherent loads: the index may come from the kernel
        // this one overlaps); the first one is also read directly, its copies start before the first barrier
        if (tid < dm.topk) ent[tid] = __ldcg(irow + tid);
        auto load_unit = [&](int m, int kb, int buf) -> bool {
            int r = m == 0 ? __ldcg(irow) : ent[m];
            const bool valid = r >= 0 && r < dm.R;
            if (!valid) { record_error(status, BRA_ERR_INDEX, r); r = 0; }
            const int qy = (r * inv_s) >> 20, qx = r - qy * dm.S;
            const size_t off = (size_t)(qy * dm.hs + kb * RT) * row_bytes + (size_t)(qx * WS) * tok_bytes;
            load_block(sm_base + OFF_KV + buf * 16384, Kb + off);
            load_block(sm_base + OFF_KV + buf * 16384 + 8192, Vb + off);
            return valid;
        };
        // ---- Q tile, V halo, first key block ----
        load_block(sm_base + OFF_Q, Qb + (size_t)y0 * row_bytes + (size_t)x0 * tok_bytes);
        if (dm.lce) {
#pragma unroll
            for (int it = 0; it < (HROWS * HCOLS * 4 + THREADS - 1) / THREADS; ++it) {
                const int q = tid + it * THREADS;
                if (q < HROWS * HCOLS * 4) {
                    const int pos = q >> 2, hy = pos / HCOLS, hx = pos - hy * HCOLS;
                    const int y = y0 - 2 + hy, x = x0 - 2 + hx;
                    const bool inb = (unsigned)y < (unsigned)dm.H && (unsigned)x < (unsigned)dm.W;
                    const uint8_t* src = inb ? Vb + (size_t)y * row_bytes + (size_t)x * tok_bytes + (q & 3) * 16 : Vb;
                    cp_async_16(sm_base + OFF_HALO + q * 16, src, inb ? 16u : 0u);
                }
            }
        }
        bool valid_next = load_unit(0, 0, 0);
        int m_next = 0, kb_next = 0;             // (routed slot, row block) of the key block being loaded
        cp_async_commit();

        // Softmax over the routed key blocks without a rescaling step per block: the first valid block
        // fixes the reference maximum m_run (its own row maximum); later blocks use it as it stands, so
        // their probabilities exp2(s - m_run) may exceed 1.  That is exact as long as nothing overflows
        // (numerator and denominator carry the same factor); a block whose row sum comes out above 2^40
        // anywhere in the CTA is done again the slow way: S recomputed, row maximum, m_run raised, the
        // sums so far rescaled.  With the maximum settled in the first block that path is rare.
        float m_run = 0.f, l_run = 0.f;
        bool have_m = false;                         // CTA-uniform: a routing entry is valid or not for the whole tile
        float o_acc[32];
#pragma unroll
        for (int q = 0; q < 32; ++q) o_acc[q] = 0.f;

        // S of a key block is made in two halves of 64 keys, columns [0,64) and [64,128) of tensor memory,
        // each with its own barrier: the low half of the NEXT block is issued right behind O = P V of this one
        // (the tensor core takes them in order, and P V is the last reader of those columns), the high half as
        // soon as every thread has read O out of columns [64,96).  So the threads never wait for an S.
        auto issue_s_half = [&](int buf, int half) {
            const uint32_t qa = sm_base + OFF_Q, ka = sm_base + OFF_KV + buf * 16384 + half * 4096;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks)           // d = 32 = 2 k-steps of 16
                umma_ss(tmem + half * 64, umma_smem_desc(qa + ks * 32, 16, 512, 4),
                        umma_smem_desc(ka + ks * 32, 16, 512, 4), IDESC_SH, ks);
            umma_commit(half ? bar_sh : bar_s);
        };
        // row maximum of S over the 128 keys of the block (raw scores), 32 columns per round trip to tensor memory
        auto block_max = [&]() -> float {
            float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll 1
            for (int cc = 0; cc < 128; cc += 32) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(tg + cc, r);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 32; q += 4) {
                    m0 = fmax3(m0, __uint_as_float(r[q]), __uint_as_float(r[q + 1]));
                    m1 = fmax3(m1, __uint_as_float(r[q + 2]), __uint_as_float(r[q + 3]));
                }
            }
            return fmaxf(m0, m1);
        };
        // P = exp2(S * scale * log2 e - m_run) for one half of the block, as bf16 pairs over columns of S
        // already consumed (half 0: [0,32), half 1: [32,64)); returns the sum over the half's 64 keys.
        // Loads from tensor memory are issued one step ahead of their use.
        auto exp_half = [&](int half) -> float {
            const float2 sl2v = make_float2(sl2, sl2), mnegv = make_float2(-m_run, -m_run);
            float2 sum2 = make_float2(0.f, 0.f);
            const uint32_t src = tg + 64 * half, dst = tg + 32 * half;
            uint32_t r[2][16];
            tmem_ld_32x32b_x16(src, r[0]);
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                tmem_ld_wait();
                if (ch < 3) tmem_ld_32x32b_x16(src + 16 * (ch + 1), r[(ch + 1) & 1]);
                uint32_t pk[8];
#pragma unroll
                for (int q = 0; q < 16; q += 2) {
                    const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[ch & 1][q]), __uint_as_float(r[ch & 1][q + 1])), sl2v, mnegv);
                    const float2 pe = make_float2(ex2w(a.x), ex2w(a.y));
                    sum2 = __fadd2_rn(sum2, pe);
                    pk[q >> 1] = packw(pe.x, pe.y);
                }
                tmem_st_32x32b_x8(dst + 8 * ch, pk);
            }
            return sum2.x + sum2.y;
        };

        // ---- first key block: wait for it (with Q), issue both halves of its S, start the copy of the second ----
        cp_async_wait<0>();
        fence_proxy_async_smem();
        if (!__syncthreads_and(ok)) { ok = false; break; }
        if (tid == 0) {
            tc_fence_after_sync();
            issue_s_half(0, 0);
            issue_s_half(0, 1);
        }
        bool valid = valid_next;
        if (units > 1) {
            if (++kb_next == RB) { kb_next = 0; ++m_next; }
            valid_next = load_unit(m_next, kb_next, 1);
            cp_async_commit();
        }

        for (int u = 0; u < units; ++u) {
            const int buf = u & 1;
            const bool more = u + 1 < units;
            float sum = 0.f;
            bool big = false;
            ok = mbar_wait(bar_s, n_s & 1, POLL_LIMIT) && ok;
            tc_fence_after_sync();
            if (valid) {
                if (!have_m) {                       // the first valid block sets the reference maximum
                    ok = mbar_wait(bar_sh, n_s & 1, POLL_LIMIT) && ok;
                    tc_fence_after_sync();
                    m_run = block_max() * sl2;       // sl2 > 0
                }
                sum = exp_half(0);
                ok = mbar_wait(bar_sh, n_s & 1, POLL_LIMIT) && ok;
                tc_fence_after_sync();
                sum += exp_half(1);
                big = !(sum <= 0x1p40f);             // also catches inf and NaN
            } else {                                 // a bad routing entry (the whole CTA sees it): P = 0
                ok = mbar_wait(bar_sh, n_s & 1, POLL_LIMIT) && ok;
                tc_fence_after_sync();
                uint32_t pk[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) pk[q] = 0u;
#pragma unroll 1
                for (int cc = 0; cc < 64; cc += 8) tmem_st_32x32b_x8(tg + cc, pk);
            }
            ++n_s;
            tmem_st_wait();
            tc_fence_before_sync();
            cp_async_wait<0>();                      // this thread's copies of block u + 1 (issued a block ago)
            fence_proxy_async_smem();
            if (__syncthreads_or(big || !ok)) {
                if (!__syncthreads_and(ok)) { ok = false; break; }   // a wait gave up somewhere: the tile ends here
                // the slow way: S again (P has overwritten its low half), true row maximum, everything rescaled
                if (tid == 0) {
                    tc_fence_after_sync();
                    issue_s_half(buf, 0);
                    issue_s_half(buf, 1);
                }
                ok = mbar_wait(bar_s, n_s & 1, POLL_LIMIT) && ok;
                ok = mbar_wait(bar_sh, n_s & 1, POLL_LIMIT) && ok;
                ++n_s;
                tc_fence_after_sync();
                const float m_new = fmaxf(m_run, block_max() * sl2);
                const float corr = ex2w(m_run - m_new);
                m_run = m_new;
                l_run *= corr;
#pragma unroll
                for (int q = 0; q < 32; ++q) o_acc[q] *= corr;
                sum = exp_half(0);
                sum += exp_half(1);
                tmem_st_wait();
                tc_fence_before_sync();
                __syncthreads();
            }
            have_m = have_m || valid;
            if (tid == 0) {
                tc_fence_after_sync();
                const uint64_t vd = umma_smem_desc(sm_base + OFF_KV + buf * 16384 + 8192, 16, 512, 4);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)       // 128 keys = 8 k-steps of 16 (1024 B of V each)
                    umma_ts(tmem + TM_O, tmem + ks * 8, vd + (uint64_t)(ks * 64), IDESC_O, ks);
                umma_commit(bar_o);
                if (more) issue_s_half(buf ^ 1, 0);  // block u + 1 has landed (the barrier above)
            }
            ok = mbar_wait(bar_o, n_o & 1, POLL_LIMIT) && ok;
            ++n_o;
            tc_fence_after_sync();
            uint32_t oraw[32];
            tmem_ld_32x32b_x32(tg + TM_O, oraw);
            tmem_ld_wait();
            tc_fence_before_sync();
            l_run += sum;
#pragma unroll
            for (int q = 0; q < 32; ++q) o_acc[q] += __uint_as_float(oraw[q]);
            if (more) {
                // columns [64,128) are free once all 128 threads have read O: the last one to say so issues the
                // high half of the next S (no barrier: the others go straight on to the low half, which is ready)
                uint32_t before;
                asm volatile("atom.acq_rel.cta.shared.add.u32 %0, [%1], 1;" : "=r"(before) : "r"(smem_u32(arrivals)) : "memory");
                if (before == n_arr * THREADS + (THREADS - 1)) {
                    tc_fence_after_sync();
                    issue_s_half(buf ^ 1, 1);
                }
                ++n_arr;
                valid = valid_next;
                if (u + 2 < units) {                 // K and V of block u are done with: block u + 2 takes their place
                    if (++kb_next == RB) { kb_next = 0; ++m_next; }
                    valid_next = load_unit(m_next, kb_next, buf);
                    cp_async_commit();
                }
            }
        }
        if (!__syncthreads_and(ok)) { ok = false; break; }   // every thread waits on the barriers itself: agree before going on

        // the head's LCE weights for this thread's channel pair: fetched here, not held through the key
        // loop (50 registers); the loads fly during the staging below
        float2 wv[25];
        float2 bias2 = make_float2(0.f, 0.f);
        if (dm.lce) {
            const float* wp = lce_w + (size_t)(h * 32 + 2 * cp) * 25;
#pragma unroll
            for (int q = 0; q < 25; ++q) wv[q] = make_float2(__ldg(wp + q), __ldg(wp + 25 + q));
        }
        if (lce_b) bias2 = make_float2(__ldg(lce_b + h * 32 + 2 * cp), __ldg(lce_b + h * 32 + 2 * cp + 1));
        // ---- normalise, stage O^att as fp32 [128 tokens][32 ch] (16-byte units xor-swizzled) ----
        {
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            const uint32_t srow = sm_base + OFF_ST + tid * 128;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                sts_f32x4(srow + ((q ^ (tid & 7)) << 4),
                          o_acc[4 * q] * inv, o_acc[4 * q + 1] * inv, o_acc[4 * q + 2] * inv, o_acc[4 * q + 3] * inv);
            if (lse)
                lse[((size_t)b * dm.heads + h) * dm.N + (size_t)(y0 + (tid >> 4)) * dm.W + x0 + (tid & 15)] =
                    (m_run + log2f(l_run)) * 0.6931471805599453f;
        }
        __syncthreads();

        // ---- LCE + store: input row yy of the halo feeds output rows yy - ti through tap row ti ----
        {
            const uint32_t halo = sm_base + OFF_HALO + xl0 * 64 + cp * 4;
            const uint32_t stage = sm_base + OFF_ST + (cp & 1) * 8;
            uint32_t* out = reinterpret_cast<uint32_t*>(O) + (img + (size_t)y0 * row_bytes + (size_t)(x0 + xl0) * tok_bytes) / 4 + cp;
            const size_t out_row = (size_t)dm.W * (dm.C / 2);
            float2 acc[RT][2];
#pragma unroll
            for (int y = 0; y < RT; ++y) { acc[y][0] = bias2; acc[y][1] = bias2; }
            if (dm.lce) {
#pragma unroll
                for (int yy = 0; yy < HROWS; ++yy) {
                    float2 v[6];
#pragma unroll
                    for (int xx = 0; xx < 6; ++xx) {
                        const uint32_t w = lds_u32(halo + (yy * HCOLS + xx) * 64);
                        v[xx] = make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
                    }
#pragma unroll
                    for (int tj = 0; tj < 5; ++tj)
#pragma unroll
                        for (int ti = 0; ti < 5; ++ti) {
                            const int y = yy - ti;
                            if (y < 0 || y >= RT) continue;
#pragma unroll
                            for (int xx = 0; xx < 2; ++xx)
                                acc[y][xx] = __ffma2_rn(wv[ti * 5 + tj], v[xx + tj], acc[y][xx]);
                        }
                }
            }
#pragma unroll
            for (int y = 0; y < RT; ++y) {
#pragma unroll
                for (int xx = 0; xx < 2; ++xx) {
                    const int tk = y * WS + xl0 + xx;
                    const float2 att = lds_f32x2(stage + tk * 128 + (((cp >> 1) ^ (tk & 7)) << 4));
                    const float2 r2 = __fadd2_rn(att, acc[y][xx]);
                    out[xx * (dm.C / 2)] = packw(r2.x, r2.y);
                }
                out += out_row;
            }
        }
        __syncthreads();                             // staging tile (over Q) and halo are free
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
bool attend_tc_wide_supported(const Dims& d, int dtype) {
    return dtype == BRA_BF16 && d.d == 32 && d.ws == tw::WS && d.hs % tw::RT == 0 && d.topk <= tw::KCAP && d.R <= 4096 &&
           (long long)d.B * d.R * d.heads * (d.hs / tw::RT) < (1ll << 30);
}

cudaError_t launch_attend_tc_wide(const Dims& d, const void* Q, const void* K, const void* V,
                                  const int32_t* index, const float* lce_w, const float* lce_b,
                                  void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel) {
    static PerDeviceOnce attr_set;
    cudaError_t e = attr_set.run([] {
        cudaError_t a = cudaFuncSetAttribute(attend_tc_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tw::SMEM_BYTES);
        if (a != cudaSuccess) return a;
        return cudaFuncSetAttribute(attend_tc_wide_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    });
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 1;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return cudaErrorUnknown;
    const int tiles = d.B * d.R * d.heads * (d.hs / tw::RT);
    const int resident = sms * 4;
    const unsigned grid = (unsigned)(tiles < resident ? tiles : resident);
    e = launch_kernel(attend_tc_wide_kernel, dim3(grid), dim3(tw::THREADS), tw::SMEM_BYTES, st,
                                  after_own_kernel,
                                  static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(K),
                                  static_cast<const __nv_bfloat16*>(V), index, lce_w, lce_b,
                                  static_cast<__nv_bfloat16*>(O), lse, status, d, tiles);
    count_launch();
    return e;
}

}  // namespace bra
