// Routed token-to-token attention + LCE on the 5th-generation tensor cores for topk = 1
// (Eq. 6, Eq. 7 with Eq. 1): every query region attends to one routed region per head, so a tile
// needs one S = Q K^T, one softmax without running maximum, and one O = P V.
//
// Tile layout and thread mappings are those of attend_tc.cu (two heads stacked into a 128-row MMA
// tile, 128-thread CTAs, four per SM).  Two things differ.
//
// Copies: the tiles reach shared memory as bulk tensor copies (TMA) issued by one thread: per tile
// two {32 ch, 8, 8} boxes each of Q, of K and of V (one per head; the gather of Eq. 6 is the box
// coordinates of the routed regions) in the 64-byte swizzled layout the MMA descriptors name, and
// one {64 ch, 12, 12} box of V around the query region for the LCE, zero-filled outside the map (the
// conv's padding).  Measured on B200 with four CTAs per SM these boxes fill shared memory at
// 10-11 TB/s against 8.5 TB/s for per-thread 16-byte copies, and cost the other 127 threads no
// address arithmetic at all.  Tensor maps cover this GPU's own memory; nothing is multicast.
//
// Schedule: the tensor core works one tile ahead of the threads.  While the threads run the softmax
// and P V of tile n, Q and K of tile n + 1 land in the buffers S_n has released; S_{n+1} = Q K^T is
// issued before the LCE of tile n starts and completes underneath it.  V of tile n + 1 follows once
// the staging tile that overlays it has been read, the halo once the LCE is done.  Per tile:
//   wait S_n  ->  copies of Q, K of tile n + 1 go out  ->  softmax, P to TMEM  ->  O = P V (two
//   MMAs, one per head's V tile)  ->  normalised O^att to the fp32 staging tile  ->  S_{n+1} issued
//   ->  LCE sums start from O^att  ->  copy of V of tile n + 1 goes out  ->  LCE (5x5 depthwise
//   correlation of V from the halo tile), one bf16 store of O  ->  copy of the halo of tile n + 1.
// Every wait (on an MMA, on a copy) is bounded.
#include "attend_tc_common.cuh"

namespace bra {

namespace k1 {
constexpr int OFF_VB = tc::OFF_V + 4096;        // head B's V tile ([64 keys][64 B], 64-byte swizzle), after head A's
constexpr uint32_t QK_BYTES = 16384, V_BYTES = 8192;
}  // namespace k1

// ------------------------------------------------------------------ the forward pass in one launch
// What the one-launch forward adds to the arguments of the attention kernel.  The grid runs three phases:
// region pooling of Q and K, routing (Eq. 4, Eq. 5 with k = 1), then the attention above.  The work of the
// first two phases is handed out by ticket counters and a phase is over when a completion counter has
// reached the number of its work items: CTAs that are running do all of it, so progress never depends on
// how many CTAs of the grid are resident (and every wait is bounded all the same).  Pooling and routing add
// their terms in the order of the stand-alone kernels, so the index equals bra_route's bit for bit.
struct FwdArgs {
    const uint8_t* Q;       // [B,H,W,C] bf16
    const uint8_t* K;
    float* q_mean;          // [B,R,C] Q^r (scratch)
    float* k_mean;          // [B,R,C] K^r (scratch)
    int32_t* index_out;     // [B,heads,R,1]
    int32_t* ctrl;          // status block; [8] pooling tickets, [9] pooled units, [10] routing tickets, [11] routed
                            // items, [12] finished CTAs: zero at launch, put back to zero by the last CTA
    int inject;             // failure injection of the tests: 1 = the first pooled unit is never counted
};

// Bounded wait until *ctr has reached target (all threads return the same answer).
__device__ __noinline__ bool wait_count(const int32_t* ctr, int target, uint32_t polls) {
    bool ok = true;
    if (threadIdx.x == 0) {
        ok = false;
        for (uint32_t it = 0; it < polls; ++it) {
            if (ld_acquire_gpu(ctr) >= target) { ok = true; break; }
            __nanosleep(it < 32 ? 20 : 200);
        }
    }
    return __syncthreads_and(ok);
}

// Phase 1: per-region average of Q and K (Section 3.2).  A unit is (image, region, 64-channel slab); thread
// (row half, column, 16-byte channel vector) sums its four token rows in order, then one thread per channel
// adds, column by column, (lower half + upper half): the order of the stand-alone kernel for 8-row regions.
// The loads of the next unit fly while this one is reduced; its ticket was drawn a unit earlier.
__device__ __noinline__ void forward_pool_phase(const FwdArgs& fw, const Dims& dm, uint8_t* smem) {
    using namespace tc;
    const int tid = threadIdx.x;
    const int c = tid & 7, tx = (tid >> 3) & 7, yh = tid >> 6;
    const int pairs = dm.heads >> 1;
    const int units = dm.B * dm.R * pairs;
    const size_t row_bytes = (size_t)dm.W * dm.C * 2;
    const uint32_t part = smem_u32(smem) + OFF_POOL;         // [tensor][row half][column][64 ch] fp32
    volatile int* slot = reinterpret_cast<volatile int*>(smem + OFF_MISC);
    auto unit_off = [&](int u) -> size_t {
        const int hp = u % pairs, r = (u / pairs) % dm.R, b = u / (pairs * dm.R);
        const int ry = r / dm.S, rx = r - ry * dm.S;
        return (size_t)b * dm.H * row_bytes + (size_t)(ry * RS + 4 * yh) * row_bytes + (size_t)(rx * RS + tx) * dm.C * 2 +
               (size_t)hp * 128 + c * 16;
    };
    auto load_unit = [&](int u, uint4 (&v)[8]) {
        const size_t off = unit_off(u);
#pragma unroll
        for (int q = 0; q < 4; ++q) { v[q] = ldg_nc_u4(fw.Q + off + q * row_bytes); v[4 + q] = ldg_nc_u4(fw.K + off + q * row_bytes); }
    };
    if (tid == 0) { slot[0] = atomicAdd(fw.ctrl + 8, 1); slot[1] = atomicAdd(fw.ctrl + 8, 1); }
    __syncthreads();
    int cur = slot[0], nxt = slot[1];
    __syncthreads();
    uint4 pv[8];
    int done = 0;                                           // units this CTA has pooled: counted in one go at the end
    if (cur < units) load_unit(cur, pv);
    while (cur < units) {
        int t2 = 0;
        if (tid == 0) t2 = atomicAdd(fw.ctrl + 8, 1);       // the unit after next
        uint4 nx[8];
        if (nxt < units) load_unit(nxt, nx);
#pragma unroll
        for (int tsr = 0; tsr < 2; ++tsr) {
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint4 v = pv[4 * tsr + q];
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    acc[2 * e] += __uint_as_float(w[e] << 16);
                    acc[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
                }
            }
            const uint32_t dst = part + ((((tsr * 2 + yh) * 8 + tx) * 64 + c * 8) << 2);
            sts_f32x4(dst, acc[0], acc[1], acc[2], acc[3]);
            sts_f32x4(dst + 16, acc[4], acc[5], acc[6], acc[7]);
        }
        __syncthreads();
        {
            const int tsr = tid >> 6, ch = tid & 63;
            const uint32_t src = part + (((tsr * 2) * 8 * 64 + ch) << 2);
            float s = 0.f;
#pragma unroll
            for (int x = 0; x < 8; ++x) s += lds_f32(src + x * 256) + lds_f32(src + 8 * 256 + x * 256);
            const int hp = cur % pairs, r = (cur / pairs) % dm.R, b = cur / (pairs * dm.R);
            float* dst = tsr ? fw.k_mean : fw.q_mean;
            dst[((size_t)b * dm.R + r) * dm.C + hp * 64 + ch] = s * (1.0f / 64.0f);
        }
        if (tid == 0) slot[0] = t2;
        __syncthreads();
        if (!(fw.inject && cur == 0)) ++done;
        cur = nxt;
        nxt = slot[0];
#pragma unroll
        for (int q = 0; q < 8; ++q) pv[q] = nx[q];
    }
    __threadfence();
    __syncthreads();
    if (tid == 0 && done) atomicAdd(fw.ctrl + 9, done);
}

// Phase 2: Eq. 4 and Eq. 5 (k = 1).  An item is (image, head, chunk of 16 affinity rows); K^r of the head
// sits in shared memory as [R][8 x 16 B] with unit (c4 + j) & 7 of row j holding channels 4 c4..4 c4+3
// (conflict-free for 16-byte reads by eight consecutive rows).  Thread = (row, one of eight candidate
// classes j mod 8); each dot product adds its 32 channels in increasing order, as the stand-alone routing
// kernels do; the best (score, lower region first) of the eight classes is found with shuffles.
__device__ __noinline__ void forward_route_phase(const FwdArgs& fw, const Dims& dm, uint8_t* smem) {
    using namespace tc;
    const int tid = threadIdx.x;
    const uint32_t ks = smem_u32(smem) + OFF_POOL;
    volatile int* slot = reinterpret_cast<volatile int*>(smem + OFF_MISC);
    const int chunks = (dm.R + 15) >> 4;
    const int items = dm.B * dm.heads * chunks;
    const int l8 = tid & 7, lrow = tid >> 3;
    for (;;) {
        if (tid == 0) slot[0] = atomicAdd(fw.ctrl + 10, 1);
        __syncthreads();
        const int it = slot[0];
        if (it >= items) break;
        const int ch = it % chunks, h = (it / chunks) % dm.heads, b = it / (chunks * dm.heads);
        const float* kb = fw.k_mean + (size_t)b * dm.R * dm.C + h * 32;
        for (int e = tid; e < dm.R * 8; e += THREADS) {
            const int j = e >> 3, c4 = e & 7;
            const float4 v = __ldcg(reinterpret_cast<const float4*>(kb + (size_t)j * dm.C) + c4);
            sts_f32x4(ks + ((j * 8 + ((c4 + j) & 7)) << 4), v.x, v.y, v.z, v.w);
        }
        const int i = ch * 16 + lrow;
        const bool live = i < dm.R;
        float4 q[8];
        {
            const float4* qrow = reinterpret_cast<const float4*>(fw.q_mean + ((size_t)b * dm.R + (live ? i : 0)) * dm.C + h * 32);
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) q[c4] = __ldcg(qrow + c4);
        }
        __syncthreads();
        unsigned long long best = 0ull;
        for (int j = l8; j < dm.R; j += 8) {
            float acc = 0.f;
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) {
                const float4 k4 = lds_f32x4(ks + ((j * 8 + ((c4 + j) & 7)) << 4));
                acc = fmaf(q[c4].x, k4.x, acc);
                acc = fmaf(q[c4].y, k4.y, acc);
                acc = fmaf(q[c4].z, k4.z, acc);
                acc = fmaf(q[c4].w, k4.w, acc);
            }
            const unsigned long long key = ((unsigned long long)score_bits(acc) << 32) | (0xffffffffu - (uint32_t)j);
            best = key > best ? key : best;
        }
#pragma unroll
        for (int sh = 1; sh < 8; sh <<= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, sh);
            best = other > best ? other : best;
        }
        if (l8 == 0 && live)
            fw.index_out[((size_t)b * dm.heads + h) * dm.R + i] = (int32_t)(0xffffffffu - (uint32_t)best);
        __threadfence();
        __syncthreads();                    // index written; K^r of the next item may take the place of this one
        if (tid == 0) atomicAdd(fw.ctrl + 11, 1);
    }
}

struct K1Maps { CUtensorMap q, k, v, halo; };   // {32 ch, 8, 8} boxes of Q, K, V; {64 ch, 12, 12} box of V

// FORWARD: pooling and routing run first, in this launch (see FwdArgs).
template <bool FORWARD>
__global__ void __launch_bounds__(tc::THREADS, 4)
attend_tc_k1_kernel(const __grid_constant__ K1Maps maps, const int32_t* index,
                    const float* __restrict__ lce_w, const float* __restrict__ lce_b,
                    __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
                    int32_t* __restrict__ status, Dims dm, int num_tiles, FwdArgs fw) {
    using namespace tc;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bar_s = reinterpret_cast<uint64_t*>(smem + OFF_BAR);       // S landed in TMEM
    uint64_t* bar_o = bar_s + 1;                                         // O landed in TMEM
    uint64_t* bar_qk = bar_s + 2;                                        // Q and K tiles landed in shared memory
    uint64_t* bar_v = bar_s + 3;                                         // V tiles landed
    uint64_t* bar_h = bar_s + 4;                                         // halo landed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_s + 5);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int inv_s = (1 << 20) / dm.S + 1;            // i / S == (i * inv_s) >> 20 for i < 4096
    const int my_tiles = (num_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (tid == 0) {
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        mbar_init(bar_qk, 1);
        mbar_init(bar_v, 1);
        mbar_init(bar_h, 1);
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    TileWalker walk;
    walk.init(blockIdx.x, gridDim.x, dm);
    const uint32_t sm_base = smem_u32(smem);

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
    // routing entries (head A, head B) of a tile; -1: out of range.  The index may come from a kernel this
    // one overlaps (programmatic dependent launch): coherent loads after pdl_wait(), never the read-only
    // path, whose loads the compiler may move above the wait
    // The loads are issued two tiles ahead of the tile they serve and looked at (checked) one tile later,
    // so that their latency is never waited for.
    auto load_entries = [&](int b, int i, int hp) -> int2 {
        const int hA = 2 * hp, hB = hA + 1;
        const int hiA = dm.heads_i == 1 ? 0 : hA, hiB = dm.heads_i == 1 ? 0 : hB;
        return make_int2(__ldcg(index + ((size_t)b * dm.heads_i + hiA) * dm.R + i),
                         __ldcg(index + ((size_t)b * dm.heads_i + hiB) * dm.R + i));
    };
    auto checked = [&](int2 e) -> int2 {
        if (e.x < 0 || e.x >= dm.R) { record_error(status, BRA_ERR_INDEX, e.x); e.x = -1; }
        if (e.y < 0 || e.y >= dm.R) { record_error(status, BRA_ERR_INDEX, e.y); e.y = -1; }
        return e;
    };
    // ---- copies: issued by thread 0 only.  A box is named by (channel, x, y, image) of its first element.
    // j: ordinal of the tile among this CTA's (its parity is the phase of the barrier); remembered so that
    // a CTA that gives up can still wait for what it has in flight.
    int last_qk = -1, last_v = -1, last_h = -1;
    auto issue_qk = [&](const TileCoord& t, int2 ent, int j) {
        last_qk = j;
        const int ra = ent.x < 0 ? 0 : ent.x, rb = ent.y < 0 ? 0 : ent.y;   // an invalid entry loads region 0; its P is zero
        const int rya = (ra * inv_s) >> 20, ryb = (rb * inv_s) >> 20;
        mbar_expect_tx(bar_qk, k1::QK_BYTES);
        tma_load_4d(sm_base + OFF_Q, &maps.q, bar_qk, t.c0, t.x0, t.y0, t.b);
        tma_load_4d(sm_base + OFF_Q + 4096, &maps.q, bar_qk, t.c0 + 32, t.x0, t.y0, t.b);
        tma_load_4d(sm_base + OFF_K, &maps.k, bar_qk, t.c0, (ra - rya * dm.S) * RS, rya * RS, t.b);
        tma_load_4d(sm_base + OFF_K + 4096, &maps.k, bar_qk, t.c0 + 32, (rb - ryb * dm.S) * RS, ryb * RS, t.b);
    };
    auto issue_v = [&](const TileCoord& t, int2 ent, int j) {
        last_v = j;
        const int ra = ent.x < 0 ? 0 : ent.x, rb = ent.y < 0 ? 0 : ent.y;
        const int rya = (ra * inv_s) >> 20, ryb = (rb * inv_s) >> 20;
        mbar_expect_tx(bar_v, k1::V_BYTES);
        tma_load_4d(sm_base + OFF_V, &maps.v, bar_v, t.c0, (ra - rya * dm.S) * RS, rya * RS, t.b);
        tma_load_4d(sm_base + k1::OFF_VB, &maps.v, bar_v, t.c0 + 32, (rb - ryb * dm.S) * RS, ryb * RS, t.b);
    };
    auto issue_halo = [&](const TileCoord& t, int j) {
        if (!dm.lce) return;
        last_h = j;
        mbar_expect_tx(bar_h, HALO_BYTES);
        tma_load_4d(sm_base + OFF_HALO, &maps.halo, bar_h, t.c0, t.x0 - 2, t.y0 - 2, t.b);
    };
    auto issue_s = [&]() {                  // S = Q K^T for the tile whose Q and K are in shared memory
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
    if (FORWARD) {
        const uint32_t polls = fw.inject ? 2048u : FLAG_POLLS;
        forward_pool_phase(fw, dm, smem);
        ok = wait_count(fw.ctrl + 9, dm.B * dm.R * (dm.heads >> 1), polls);
        if (ok) {
            forward_route_phase(fw, dm, smem);
            ok = wait_count(fw.ctrl + 11, dm.B * dm.heads * ((dm.R + 15) >> 4), polls);
        }
    } else {
        // Q and the halo are inputs of the call: their copies overlap the tail of the kernel before (routing,
        // in a forward call); only the routing index, hence K and V, has to wait for it
        if (tid == 0 && my_tiles > 0) {
            mbar_expect_tx_only(bar_qk, k1::QK_BYTES / 2);
            tma_load_4d(sm_base + OFF_Q, &maps.q, bar_qk, t.c0, t.x0, t.y0, t.b);
            tma_load_4d(sm_base + OFF_Q + 4096, &maps.q, bar_qk, t.c0 + 32, t.x0, t.y0, t.b);
            issue_halo(t, 0);
        }
        pdl_wait();                         // the routing index comes from the kernel before
    }
    int2 ent = make_int2(0, 0);             // routing entries (head A, head B) of the tile in hand
    int2 raw_n = make_int2(0, 0);           // those of the next tile, as loaded (not yet looked at)
    const int run_tiles = ok ? my_tiles : 0;    // a barrier that gave up: no tile is started
    if (my_tiles > 1) {
        walk.next();                        // the walker stays one tile ahead of `tn`
        raw_n = load_entries(walk.b, walk.i, walk.hp);
    }
    TileCoord tn = my_tiles > 1 ? coord_of(walk.b, walk.i, walk.hp) : t;
    if (run_tiles > 0) {
        ent = checked(load_entries(t.b, t.i, t.hp));
        if (tid == 0) {
            if (FORWARD) {
                issue_qk(t, ent, 0);
                issue_halo(t, 0);
            } else {                            // Q and the halo are on their way already: K completes the phase
                const int ra = ent.x < 0 ? 0 : ent.x, rb = ent.y < 0 ? 0 : ent.y;
                const int rya = (ra * inv_s) >> 20, ryb = (rb * inv_s) >> 20;
                last_qk = 0;
                mbar_expect_tx(bar_qk, k1::QK_BYTES / 2);
                tma_load_4d(sm_base + OFF_K, &maps.k, bar_qk, t.c0, (ra - rya * dm.S) * RS, rya * RS, t.b);
                tma_load_4d(sm_base + OFF_K + 4096, &maps.k, bar_qk, t.c0 + 32, (rb - ryb * dm.S) * RS, ryb * RS, t.b);
            }
            issue_v(t, ent, 0);
            ok = mbar_wait(bar_qk, 0, POLL_LIMIT);
            if (ok) issue_s();
        }
    }

    for (int n = 0; n < run_tiles; ++n) {
        if (dm.lce && t.hp != hp_loaded) {
            const float* wp = lce_w + (size_t)(t.c0 + 2 * lane) * 25;
#pragma unroll
            for (int q = 0; q < 25; ++q) wv[q] = make_float2(__ldg(wp + q), __ldg(wp + 25 + q));
            if (lce_b) bias2 = make_float2(__ldg(lce_b + t.c0 + 2 * lane), __ldg(lce_b + t.c0 + 2 * lane + 1));
            hp_loaded = t.hp;
        }
        const bool has_next = n + 1 < my_tiles;
        const int2 ent_n = has_next ? checked(raw_n) : ent;       // loaded a tile ago
        if (n + 2 < my_tiles) {
            walk.next();
            raw_n = load_entries(walk.b, walk.i, walk.hp);         // for the tile after next
        }
        const uint32_t par = n & 1;

        // ---- S of this tile is in TMEM (issued a tile ago); the MMA has read Q and K, so the next
        // tile's take their place ----
        ok = mbar_wait(bar_s, par, POLL_LIMIT) && ok;
        tc_fence_after_sync();
        if (tid == 0 && has_next && ok) issue_qk(tn, ent_n, n + 1);

        // ---- softmax: thread = row.  Loads from tensor memory are issued one step ahead of their use.
        // Pass 1: row maximum, 32 columns at a time ----
        const bool valid = (head_half ? ent.y : ent.x) >= 0;
        float mx;
        {
            float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t ra[32];
                tmem_ld_32x32b_x32(s_addr + 32 * half, ra);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 32; q += 4) {
                    m0 = fmax3(m0, __uint_as_float(ra[q]), __uint_as_float(ra[q + 1]));
                    m1 = fmax3(m1, __uint_as_float(ra[q + 2]), __uint_as_float(ra[q + 3]));
                }
            }
            mx = fmaxf(m0, m1) * sl2;                                  // sl2 > 0
        }
        // an out-of-range routing entry: every probability of the row is exp2(-inf) = 0
        const float mneg = valid ? -mx : -INFINITY;
        // pass 2: P = exp2(S * scale * log2 e - max), bf16 pairs written over the columns
        // of S already consumed (column j of P never outruns column 2j of S); row sum
        const float2 sl2v = make_float2(valid ? sl2 : 0.f, valid ? sl2 : 0.f), mnegv = make_float2(mneg, mneg);
        float2 sum2 = make_float2(0.f, 0.f);
        {
            uint32_t r[2][16];
            tmem_ld_32x32b_x16(s_addr, r[0]);
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                tmem_ld_wait();
                if (ch < 3) tmem_ld_32x32b_x16(s_addr + 16 * (ch + 1), r[(ch + 1) & 1]);
                uint32_t pk[8];
#pragma unroll
                for (int q = 0; q < 16; q += 2) {
                    const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[ch & 1][q]), __uint_as_float(r[ch & 1][q + 1])), sl2v, mnegv);
                    const float2 pe = make_float2(ex2f(a.x), ex2f(a.y));
                    sum2 = __fadd2_rn(sum2, pe);
                    pk[q >> 1] = pack_bf16(pe.x, pe.y);
                }
                tmem_st_32x32b_x8(p_addr + 8 * ch, pk);
            }
        }
        tmem_st_wait();
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) { ok = false; break; }
        // ---- O = P V: head A's V tile gives columns 64..95, head B's 96..127; a row keeps its own head's ----
        if (tid == 0) {
            ok = mbar_wait(bar_v, par, POLL_LIMIT);
            if (ok) {
                tc_fence_after_sync();
                // one B operand of N = 64 channels: head A's V tile and, 4096 bytes on (the leading-dimension
                // stride between the two 32-channel atoms), head B's
                const uint64_t vd = umma_smem_desc(sm_base + OFF_V, k1::OFF_VB - OFF_V, 512, 4);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)         // 64 keys = 4 k-steps of 16 (1024 B of a V tile each)
                    umma_ts(tmem + TM_O, tmem + ks * 8, vd + (uint64_t)(ks * 64), IDESC_O, ks);
                umma_commit(bar_o);
            }
        }
        ok = mbar_wait(bar_o, par, POLL_LIMIT) && ok;
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
        // TMEM has been read: the tensor core starts on the next tile as soon as its Q and K have landed
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) { ok = false; break; }
        if (tid == 0 && has_next) {
            ok = mbar_wait(bar_qk, par ^ 1, POLL_LIMIT);
            if (ok) issue_s();
        }

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
            // the staging tile has been read (by ordinary loads: fence before the bulk copy that overwrites
            // it): V of the next tile takes its place
            fence_proxy_async_smem();
            __syncthreads();
            if (tid == 0 && has_next && ok) issue_v(tn, ent_n, n + 1);
            if (dm.lce) {
                ok = mbar_wait(bar_h, par, POLL_LIMIT) && ok;      // the halo of this tile has landed
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
        fence_proxy_async_smem();
        __syncthreads();                    // the halo has been read: the next tile's takes its place
        if (tid == 0 && has_next && ok) issue_halo(tn, n + 1);
        t = tn;
        ent = ent_n;
        if (n + 2 < my_tiles) tn = coord_of(walk.b, walk.i, walk.hp);
    }

    // ---- teardown: nothing in flight, TMEM returned ----
    tc_fence_before_sync();
    const bool all_ok = __syncthreads_and(ok);
    if (tid == 0 && !all_ok) {
        record_error(status, BRA_ERR_TIMEOUT, blockIdx.x);
        // bounded waits for the copies this CTA still has in flight (immediate for those that have landed)
        if (last_qk >= 0) mbar_wait(bar_qk, last_qk & 1, POLL_LIMIT);
        if (last_v >= 0) mbar_wait(bar_v, last_v & 1, POLL_LIMIT);
        if (last_h >= 0) mbar_wait(bar_h, last_h & 1, POLL_LIMIT);
    }
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem, TMEM_COLS);
    }
    if (FORWARD && tid == 0) {
        // the last CTA to finish puts the counters back to zero for the next call
        __threadfence();
        if (atomicAdd(fw.ctrl + 12, 1) == (int)gridDim.x - 1 && all_ok) {
#pragma unroll
            for (int q = 8; q <= 12; ++q) fw.ctrl[q] = 0;
        }
    }
}

// ------------------------------------------------------------------ host side
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's encoder, looked up through the runtime (the library does not link against the driver).
EncodeTiledFn encoder() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Tensor map over a [B,H,W,C] bf16 tensor of this GPU's memory; box = (bc channels, bx, by tokens, 1 image).
bool make_map(CUtensorMap* m, const void* base, const Dims& d, int bc, int bx, int by, CUtensorMapSwizzle sw) {
    EncodeTiledFn enc = encoder();
    if (!enc) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)d.C, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.B};
    const cuuint64_t strides[3] = {(cuuint64_t)d.C * 2, (cuuint64_t)d.W * d.C * 2, (cuuint64_t)d.H * d.W * d.C * 2};
    const cuuint32_t box[4] = {(cuuint32_t)bc, (cuuint32_t)bx, (cuuint32_t)by, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
}  // namespace

static cudaError_t k1_attributes() {
    static PerDeviceOnce once;
    return once.run([]() -> cudaError_t {
        cudaError_t a;
        if ((a = cudaFuncSetAttribute(attend_tc_k1_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_K1)) != cudaSuccess) return a;
        if ((a = cudaFuncSetAttribute(attend_tc_k1_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_K1)) != cudaSuccess) return a;
        // several CTAs per SM: ask for the largest shared-memory carve-out
        if ((a = cudaFuncSetAttribute(attend_tc_k1_kernel<false>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess) return a;
        return cudaFuncSetAttribute(attend_tc_k1_kernel<true>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    });
}

static bool k1_maps(K1Maps* maps, const Dims& d, const void* Q, const void* K, const void* V) {
    return make_map(&maps->q, Q, d, 32, tc::RS, tc::RS, CU_TENSOR_MAP_SWIZZLE_64B) &&
           make_map(&maps->k, K, d, 32, tc::RS, tc::RS, CU_TENSOR_MAP_SWIZZLE_64B) &&
           make_map(&maps->v, V, d, 32, tc::RS, tc::RS, CU_TENSOR_MAP_SWIZZLE_64B) &&
           make_map(&maps->halo, V, d, 64, tc::HALO, tc::HALO, CU_TENSOR_MAP_SWIZZLE_NONE);
}

cudaError_t launch_attend_tc_k1(const Dims& d, const void* Q, const void* K, const void* V,
                                const int32_t* index, const float* lce_w, const float* lce_b,
                                void* O, float* lse, int32_t* status, cudaStream_t st, bool after_own_kernel) {
    cudaError_t e = k1_attributes();
    if (e != cudaSuccess) return e;
    K1Maps maps;
    if (!k1_maps(&maps, d, Q, K, V)) return cudaErrorInvalidValue;
    const int tiles = d.B * d.R * (d.heads / 2);
    const int resident = tc_sm_count() * 4;
    const unsigned grid = (unsigned)(tiles < resident ? tiles : resident);
    e = launch_kernel(attend_tc_k1_kernel<false>, dim3(grid), dim3(tc::THREADS), tc::SMEM_K1, st, after_own_kernel,
                      maps, index, lce_w, lce_b, static_cast<__nv_bfloat16*>(O), lse, status, d, tiles, FwdArgs{});
    count_launch();
    return e;
}

// The forward pass in one launch: per-head routing with k = 1, at most 64 regions, and a channel
// count for which the stand-alone pooling kernel sums in the same order (so that the index equals bra_route's).
bool forward_tc_supported(const Dims& d, int dtype) {
    return attend_tc_supported(d, dtype) && d.topk == 1 && d.heads_i == d.heads && d.R <= 64 && d.C <= 128;
}

cudaError_t launch_forward_tc(const Dims& d, const void* Q, const void* K, const void* V,
                              const float* lce_w, const float* lce_b, void* O, int32_t* index, float* lse,
                              float* q_mean, float* k_mean, int32_t* ctrl, int inject, cudaStream_t st) {
    cudaError_t e = k1_attributes();
    if (e != cudaSuccess) return e;
    K1Maps maps;
    if (!k1_maps(&maps, d, Q, K, V)) return cudaErrorInvalidValue;
    const int tiles = d.B * d.R * (d.heads / 2);
    const int resident = tc_sm_count() * 4;
    const unsigned grid = (unsigned)(tiles < resident ? tiles : resident);
    FwdArgs fw;
    fw.Q = static_cast<const uint8_t*>(Q); fw.K = static_cast<const uint8_t*>(K);
    fw.q_mean = q_mean; fw.k_mean = k_mean; fw.index_out = index; fw.ctrl = ctrl; fw.inject = inject;
    e = launch_kernel(attend_tc_k1_kernel<true>, dim3(grid), dim3(tc::THREADS), tc::SMEM_K1, st, false,
                      maps, static_cast<const int32_t*>(index), lce_w, lce_b, static_cast<__nv_bfloat16*>(O), lse, ctrl, d,
                      tiles, fw);
    count_launch();
    return e;
}

}  // namespace bra
