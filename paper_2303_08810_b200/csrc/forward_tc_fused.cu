// Algorithm 1 from the projected Q, K, V on in ONE launch, for the shapes of the topk = 1 tcgen05 kernel
// (head dim 32, regions of 8 x 8 tokens, heads in pairs): region pooling, Eq. 4, Eq. 5 and the routed
// attention + LCE of Eq. 7 as numbered jobs of one persistent grid.  Opt-in (BRA_IMPL_TC_FUSED).
//
// The CTAs draw numbered jobs from a counter.  Job t = (image slot s, unit u = (region, head pair))
// pools unit u of image s (the per-region average of Q and K, summed in the order of the stand-alone
// pooling kernel) and attends unit u of image s - delta (the tile procedure of attend_tc.cu with one
// routed step).  The CTA that completes an image's pooling also routes it (Eq. 4 and Eq. 5 for every
// region and head, in the order of the stand-alone routing kernels: the index is bit-identical) and
// raises the image's flag; attention jobs wait on that flag.  A wait only ever depends on jobs with
// smaller numbers, and a job's pooling part never waits, so the scheme cannot deadlock whatever the
// number of resident CTAs; every wait is bounded all the same.
//
// Measured on B200 at the stage-1 shape this is slower than the chain of three launches: an image's
// attention cannot start before all of its 49 regions are pooled and routed, the grid holds twelve
// images' worth of tiles at any time and the whole call is only about five tiles per CTA long, so the
// look-ahead the scheme needs (pooling -> routing -> index -> K copy) is a large part of the batch.
#include "attend_tc_common.cuh"

namespace bra {

// Fused forward: Eq. 4 + Eq. 5 (k = 1) for every region and head of image b, by the whole CTA; then the
// image's flag goes up.  Kept out of line: it runs once per image and must not weigh on the register
// allocation of the tile loop.
__device__ __noinline__ void route_image(const FusedArgs& fa, const Dims& dm, int b, uint8_t* smem) {
    using namespace tc;
    const int tid = threadIdx.x;
    const uint32_t sm_base = smem_u32(smem);
    // K^r of one head sits in the 8 KB scratch as [R][8 x 16 B], unit (c4 + j) & 7 of row j holding channels 4 c4..4 c4+3 (conflict-free
    // for 16-byte reads by consecutive rows); thread = (row i, half of the candidates), four candidates
    // at a time (independent chains; each dot product adds its channels in increasing order).
    const uint32_t ks = sm_base + OFF_POOL;
    unsigned long long* best_slot = reinterpret_cast<unsigned long long*>(smem + OFF_MISC);
    const int i = tid & 63, half = tid >> 6;
    const int jmid = (dm.R + 1) >> 1;
    const int j0 = half ? jmid : 0, j1 = half ? dm.R : jmid;
    const int nchunk = dm.R * 8;
    float4 kst[4];                                   // this thread's part of K^r of the head to come
    auto fetch_k = [&](int h) {
        const float* kb = fa.k_mean + (size_t)b * dm.R * dm.C + h * 32;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int e = tid + u * THREADS;
            if (e < nchunk) kst[u] = __ldcg(reinterpret_cast<const float4*>(kb + (size_t)(e >> 3) * dm.C) + (e & 7));
        }
    };
    fetch_k(0);
    for (int h = 0; h < dm.heads; ++h) {
        float4 q[8];
        if (i < dm.R) {
            const float4* qrow = reinterpret_cast<const float4*>(fa.q_mean + ((size_t)b * dm.R + i) * dm.C + h * 32);
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) q[c4] = __ldcg(qrow + c4);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int e = tid + u * THREADS;
            const int j = e >> 3, c4 = e & 7;
            if (e < nchunk) sts_f32x4(ks + ((j * 8 + ((c4 + j) & 7)) << 4), kst[u].x, kst[u].y, kst[u].z, kst[u].w);
        }
        __syncthreads();
        if (h + 1 < dm.heads) fetch_k(h + 1);
        if (i < dm.R) {
            unsigned long long best = 0ull;
            for (int j = j0; j < j1; j += 4) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                int jj[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) jj[e] = j + e < j1 ? j + e : j1 - 1;
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float4 k4 = lds_f32x4(ks + ((jj[e] * 8 + ((c4 + jj[e]) & 7)) << 4));
                        acc[e] = fmaf(q[c4].x, k4.x, acc[e]);
                        acc[e] = fmaf(q[c4].y, k4.y, acc[e]);
                        acc[e] = fmaf(q[c4].z, k4.z, acc[e]);
                        acc[e] = fmaf(q[c4].w, k4.w, acc[e]);
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {        // a clamped repeat of the last candidate changes nothing
                    const unsigned long long key = ((unsigned long long)score_bits(acc[e]) << 32) | (0xffffffffu - (uint32_t)jj[e]);
                    best = key > best ? key : best;
                }
            }
            best_slot[half * 64 + i] = best;
        }
        __syncthreads();
        if (tid < dm.R) {
            const unsigned long long a = best_slot[tid], bb = best_slot[64 + tid];
            const unsigned long long top = a > bb ? a : bb;
            fa.index_out[((size_t)b * dm.heads + h) * dm.R + tid] = (int32_t)(0xffffffffu - (uint32_t)top);
        }
        // (the scratch is rewritten only after this barrier, best_slot only after the next head's first one)
    }
    __threadfence();
    __syncthreads();
    if (tid == 0 && !fa.inject) st_release_gpu(fa.route_flag + b, 1);
}

__global__ void __launch_bounds__(tc::THREADS, 4)
forward_tc_fused_kernel(const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ Kg,
                 const __nv_bfloat16* __restrict__ Vg, const int32_t* index,
                 const float* __restrict__ lce_w, const float* __restrict__ lce_b,
                 __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
                 int32_t* __restrict__ status, Dims dm, int num_tiles, FusedArgs fa) {
    using namespace tc;
    constexpr bool K1 = true, FUSED = true;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bar_s = reinterpret_cast<uint64_t*>(smem + OFF_BAR);       // S landed in TMEM
    uint64_t* bar_o = bar_s + 1;                                         // O landed in TMEM
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_s + 2);
    int* last_slot = reinterpret_cast<int*>(tmem_slot + 1);              // fused: "this CTA routes the image"
    int4* job_slot = reinterpret_cast<int4*>(smem + OFF_BAR + 32);       // fused: two decoded jobs

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int k = K1 ? 1 : dm.topk;
    const int pairs = dm.heads >> 1;
    const int inv_s = (1 << 20) / dm.S + 1;            // i / S == (i * inv_s) >> 20 for i < 4096

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
    // The weights of a channel pair stay in registers from tile to tile; the fused forward, which needs
    // the registers for the pooling loads in flight, fetches them again (cache hits) before each LCE.
    const int xl0 = 2 * warp;
    float2 wv_keep[25];
#pragma unroll
    for (int q = 0; q < 25; ++q) wv_keep[q] = make_float2(0.f, 0.f);
    float2 bias_keep = make_float2(0.f, 0.f);
    int hp_loaded = -1;

    constexpr uint32_t IDESC_S = umma_idesc_bf16(128, 128, false, false);
    constexpr uint32_t IDESC_O = umma_idesc_bf16(128, 64, false, true);

    bool ok = true;
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
    // come from a kernel this one overlaps (programmatic dependent launch) or, in the fused forward,
    // from another CTA of this launch: coherent loads after the wait, never the read-only path
    auto index_entries = [&](const TileCoord& t, int m) -> int2 {
        const int hA = 2 * t.hp, hB = hA + 1;
        const int hiA = dm.heads_i == 1 ? 0 : hA, hiB = dm.heads_i == 1 ? 0 : hB;
        int ra = __ldcg(index + (((size_t)t.b * dm.heads_i + hiA) * dm.R + t.i) * dm.topk + m);
        int rb = __ldcg(index + (((size_t)t.b * dm.heads_i + hiB) * dm.R + t.i) * dm.topk + m);
        return make_int2(ra, rb);
    };
    auto checked = [&](int2 e) -> int2 {
        if (e.x < 0 || e.x >= dm.R) { record_error(status, BRA_ERR_INDEX, e.x); e.x = -1; }
        if (e.y < 0 || e.y >= dm.R) { record_error(status, BRA_ERR_INDEX, e.y); e.y = -1; }
        return e;
    };
    // fused forward: bounded wait until the image of tile t has been routed
    auto wait_routed = [&](const TileCoord& t) -> bool {
        const int32_t* flag = fa.route_flag + t.b;
        const uint32_t limit = fa.inject ? 2048u : FLAG_POLLS;
        for (uint32_t it = 0; it < limit; ++it) {
            if (ld_acquire_gpu(flag) != 0) return true;
            __nanosleep(it < 64 ? 32 : 256);
        }
        record_error(status, BRA_ERR_TIMEOUT, t.b);
        ok = false;
        return false;
    };
    auto read_entries = [&](const TileCoord& t, int m) -> int2 {
        if (FUSED && !wait_routed(t)) return make_int2(-1, -1);
        return checked(index_entries(t, m));
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

    // ---- fused forward: pooling of one unit, and the routing of an image -------------------------------
    // Pooling mirrors the stand-alone kernel for regions eight rows high: thread (row half yh, column tx,
    // 16-byte channel vector c) sums its four token rows in order; then one thread per channel adds, column
    // by column, (lower half + upper half).  The loader mapping above is exactly that thread grid.
    auto pool_issue = [&](const Job& jb, uint4 (&pv)[8]) {
        const size_t off = region_off(jb.pool_b, jb.i, jb.hp * 64);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            pv[u] = ldg_nc_u4(Qb + off + u * row_bytes);
            pv[4 + u] = ldg_nc_u4(Kb + off + u * row_bytes);
        }
    };
    auto pool_finish = [&](const Job& jb, const uint4 (&pv)[8]) {
        const uint32_t part = sm_base + OFF_POOL;        // [tensor][row half][column][64 ch] fp32
#pragma unroll
        for (int tsr = 0; tsr < 2; ++tsr) {
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint4 v = pv[4 * tsr + u];
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    acc[2 * e] += __uint_as_float(w[e] << 16);
                    acc[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
                }
            }
            const uint32_t dst = part + ((((tsr * 2 + head_half) * 8 + tx) * 64 + c * 8) << 2);
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
            float* dst = tsr ? fa.k_mean : fa.q_mean;
            dst[((size_t)jb.pool_b * dm.R + jb.i) * dm.C + jb.hp * 64 + ch] = s * (1.0f / 64.0f);
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int done = atomicAdd(fa.pool_cnt + jb.pool_b, 1) + 1;
            if (done == fa.units) __threadfence();
            *last_slot = done == fa.units;
        }
        __syncthreads();
        if (*last_slot) route_image(fa, dm, jb.pool_b, smem);
    };
    auto decode_job = [&](int ticket) -> int4 {
        int4 j = make_int4(-1, -1, 0, 0);
        if (ticket < fa.total) {
            const int s = ticket / fa.units, u = ticket - s * fa.units;
            j.x = s >= fa.delta ? s - fa.delta : -1;
            j.y = s < dm.B ? s : -1;
            j.z = u / pairs;
            j.w = u - j.z * pairs;
        }
        return j;
    };

    // ---- the jobs of this CTA ---------------------------------------------------------------------------
    uint32_t n_s = 0, n_o = 0;              // uses of bar_s / bar_o so far (phase parity)
    TileWalker walk;
    int tiles_left = 0;
    Job cur, nxt;
    if (FUSED) {
        if (tid == 0) {
            if (blockIdx.x == 0) { fa.ctrl[2] = fa.sync_off; fa.ctrl[3] = fa.sync_bytes; }
            const int t0 = atomicAdd(fa.ctrl + 8, 1), t1 = atomicAdd(fa.ctrl + 8, 1);
            job_slot[0] = decode_job(t0);
            job_slot[1] = decode_job(t1);
        }
        __syncthreads();
        const int4 a = job_slot[0], bq = job_slot[1];
        cur = Job{a.x, a.y, a.z, a.w};
        nxt = Job{bq.x, bq.y, bq.z, bq.w};
        __syncthreads();
    } else {
        walk.init(blockIdx.x, gridDim.x, dm);
        tiles_left = (num_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
        cur = Job{tiles_left > 0 ? walk.b : -1, -1, walk.i, walk.hp};
        if (tiles_left > 1) { walk.next(); nxt = Job{walk.b, -1, walk.i, walk.hp}; }
        else nxt = Job{-1, -1, 0, 0};
    }
    // copies of a tile go out in two groups: (Q, K of the first routed step), then (V, halo)
    int2 ent = make_int2(0, 0);             // entries of the unit whose K/V are being loaded
    auto issue_tile = [&](const TileCoord& t, bool have_entries) {
        load_q(t);
        if (!have_entries) ent = read_entries(t, 0);
        load_k(t, ent, 0);
        cp_async_commit();
        load_v(t, ent, 0);
        load_halo(t);
        cp_async_commit();
    };
    if (cur.att_b >= 0) {
        const TileCoord t = coord_of(cur.att_b, cur.i, cur.hp);
        if (FUSED) {
            issue_tile(t, false);
        } else {
            // Q and the V halo are inputs of the call: their copies (and everything above) overlap the tail
            // of the kernel before (routing, in a forward call); only the routing index has to wait for it
            load_q(t);
            pdl_wait();
            ent = read_entries(t, 0);
            load_k(t, ent, 0);
            cp_async_commit();
            load_v(t, ent, 0);
            load_halo(t);
            cp_async_commit();
        }
    } else if (!FUSED) {
        pdl_wait();
    }

    int n = 0;
    while (cur.att_b >= 0 || cur.pool_b >= 0) {
        int ticket2 = 0;
        if (FUSED && tid == 0) ticket2 = atomicAdd(fa.ctrl + 8, 1);      // the job after next
        uint4 pv[8];
        const bool has_next = nxt.att_b >= 0;
        const TileCoord tn = coord_of(has_next ? nxt.att_b : 0, nxt.i, nxt.hp);

        if (cur.att_b >= 0) {
            const TileCoord t = coord_of(cur.att_b, cur.i, cur.hp);
            if (!FUSED && dm.lce && t.hp != hp_loaded) {
                const float* wp = lce_w + (size_t)(t.c0 + 2 * lane) * 25;
#pragma unroll
                for (int q = 0; q < 25; ++q) wv_keep[q] = make_float2(__ldg(wp + q), __ldg(wp + 25 + q));
                if (lce_b) bias_keep = make_float2(__ldg(lce_b + t.c0 + 2 * lane), __ldg(lce_b + t.c0 + 2 * lane + 1));
                hp_loaded = t.hp;
            }
            float m_run = -INFINITY, l_run = 0.f;
            bool next_routed = true;
            float o_acc[32];
#pragma unroll
            for (int q = 0; q < 32; ++q) o_acc[q] = 0.f;
            for (int m = 0; m < k; ++m) {
                const int buf = K1 ? 0 : (m & 1);
                const int2 ent_cur = ent;
                // ---- Q and this step's K have landed; make them visible to the tensor core ----
                if (m == 0) cp_async_wait<1>(); else cp_async_wait<0>();
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
                // ---- fused forward: this job's pooling (and, once per image, its routing) while S is formed;
                // before any wait on a flag, so that a wait only ever depends on jobs numbered below its own ----
                if (FUSED && m == 0 && cur.pool_b >= 0) {
                    pool_issue(cur, pv);
                    pool_finish(cur, pv);
                }
                // ---- next routed step of this tile: K/V into the other buffer (its MMAs are done) ----
                const bool more = !K1 && m + 1 < k;
                if (more) {
                    ent = read_entries(t, m + 1);
                    load_k(t, ent, buf ^ 1);
                    load_v(t, ent, buf ^ 1);
                    cp_async_commit();
                } else if (has_next) {
                    // in flight during the softmax.  Fused forward: a look only; the image may not be routed
                    // yet, in which case the entries are read again after the last MMA of this tile
                    if (FUSED) next_routed = ld_acquire_gpu(fa.route_flag + tn.b) != 0;
                    ent = index_entries(tn, 0);
                }
                const bool valid = (head_half ? ent_cur.y : ent_cur.x) >= 0;
                if (warp == 0) ok = mbar_wait(bar_s, n_s & 1, POLL_LIMIT) && ok;   // one warp polls, the rest sleep at the barrier
                ++n_s;
                if (!__syncthreads_and(ok)) { ok = false; break; }
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
                // this step's V has landed (first step: the group of V and the halo, which leaves the copies
                // of the next routed step, if any, in flight)
                if (m == 0) {
                    if (more) cp_async_wait<1>(); else cp_async_wait<0>();
                    fence_proxy_async_smem();
                }
                tc_fence_before_sync();
                __syncthreads();
                if (tid == 0) {
                    tc_fence_after_sync();
                    const uint64_t vd = umma_smem_desc(sm_base + (buf ? OFF_KV1 + 8192 : OFF_V), 16, 1024, 2);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)         // 64 keys = 4 k-steps of 16 (2048 B of V each)
                        umma_ts(tmem + TM_O, tmem + ks * 8, vd + (uint64_t)(ks * 128), IDESC_O, ks);
                    umma_commit(bar_o);
                }
                if (warp == 0) ok = mbar_wait(bar_o, n_o & 1, POLL_LIMIT) && ok;
                ++n_o;
                if (!__syncthreads_and(ok)) { ok = false; break; }
                tc_fence_after_sync();
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

            // every MMA of this tile has read its operands: Q and K (buffer 0) of the next tile go out now
            if (has_next) {
                load_q(tn);
                if (FUSED && !next_routed) ent = wait_routed(tn) ? index_entries(tn, 0) : make_int2(-1, -1);
                ent = checked(ent);
                load_k(tn, ent, 0);
            }
            cp_async_commit();
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
            __syncthreads();

            // ---- LCE + store ----
            // Input row yy of the halo feeds output rows yy - ti through tap row ti.  Fully unrolled:
            // the 8 x 2 output sums of this thread's channel pair sit in registers under fixed names,
            // starting from O^att (+ bias).
            {
                const uint32_t halo = sm_base + OFF_HALO + (xl0 * 32 + lane) * 4;
                const uint32_t stage = sm_base + OFF_ST + xl0 * 256 + (lane & 1) * 8;
                uint32_t* out = reinterpret_cast<uint32_t*>(O) +
                                ((((size_t)t.b * dm.H + t.y0) * dm.W + t.x0 + xl0) * dm.C + t.c0) / 2 + lane;
                const size_t out_row = (size_t)dm.W * (dm.C / 2);
                // staging token tk = y * 8 + xl0 + xx: its 16-byte unit index is xor-ed with tk & 7
                const uint32_t sw0 = (((lane >> 1) ^ (xl0 & 7)) << 4), sw1 = (((lane >> 1) ^ ((xl0 + 1) & 7)) << 4);
                float2 wv[25];
                float2 bias2 = bias_keep;
                if (FUSED) {
                    if (dm.lce) {
                        const float* wp = lce_w + (size_t)(t.c0 + 2 * lane) * 25;
#pragma unroll
                        for (int q = 0; q < 25; ++q) wv[q] = make_float2(__ldg(wp + q), __ldg(wp + 25 + q));
                        if (lce_b) bias2 = make_float2(__ldg(lce_b + t.c0 + 2 * lane), __ldg(lce_b + t.c0 + 2 * lane + 1));
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < 25; ++q) wv[q] = wv_keep[q];
                }
                float2 acc[8][2];
#pragma unroll
                for (int y = 0; y < 8; ++y)
#pragma unroll
                    for (int xx = 0; xx < 2; ++xx)
                        acc[y][xx] = __fadd2_rn(lds_f32x2(stage + (y * RS + xx) * 256 + (xx ? sw1 : sw0)), bias2);
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
#pragma unroll
                for (int y = 0; y < 8; ++y) {
#pragma unroll
                    for (int xx = 0; xx < 2; ++xx) out[xx * (dm.C / 2)] = pack_bf16(acc[y][xx].x, acc[y][xx].y);
                    out += out_row;
                }
            }
        } else {
            // a job without an attention part (the first delta image slots): pooling only
            pool_issue(cur, pv);
            pool_finish(cur, pv);
        }
        if (FUSED && tid == 0) job_slot[n & 1] = decode_job(ticket2);
        __syncthreads();                    // staging tile (over V) and halo are free
        if (cur.att_b >= 0) {
            if (has_next) { load_v(tn, ent, 0); load_halo(tn); }
            cp_async_commit();
        } else {
            if (has_next) issue_tile(tn, false); else { cp_async_commit(); }
        }
        cur = nxt;
        if (FUSED) {
            const int4 a = job_slot[n & 1];
            nxt = Job{a.x, a.y, a.z, a.w};
        } else {
            --tiles_left;
            if (tiles_left > 1) { walk.next(); nxt = Job{walk.b, -1, walk.i, walk.hp}; }
            else nxt = Job{-1, -1, 0, 0};
        }
        ++n;
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
    if (FUSED) {
        // the last CTA to finish puts the counters and flags back to zero for the next call
        if (tid == 0) {
            __threadfence();
            *last_slot = atomicAdd(fa.ctrl + 9, 1) == (int)gridDim.x - 1;
        }
        __syncthreads();
        if (*last_slot && ok) {
            for (int e = tid; e < dm.B; e += THREADS) { fa.pool_cnt[e] = 0; fa.route_flag[e] = 0; }
            if (tid == 0) { fa.ctrl[8] = 0; fa.ctrl[9] = 0; }
        }
    }
}

// ------------------------------------------------------------------ host side
// Per-head routing with k = 1, at most 64 regions, and a channel count for which the stand-alone pooling
// kernel sums in the same order (so that the result equals bra_route's bit for bit).
bool forward_tc_supported(const Dims& d, int dtype) {
    return attend_tc_supported(d, dtype) && d.topk == 1 && d.heads_i == d.heads && d.R <= tc::FUSED_MAX_R &&
           d.C <= 128 && ((long long)d.B + 64) * d.R * (d.heads / 2) < (1ll << 30);
}

cudaError_t launch_forward_tc(const Dims& d, const void* Q, const void* K, const void* V,
                              const float* lce_w, const float* lce_b, void* O, int32_t* index, float* lse,
                              float* q_mean, float* k_mean, int32_t* ctrl, int32_t* sync, int inject,
                              cudaStream_t st) {
    static PerDeviceOnce once;
    cudaError_t e = once.run([]() -> cudaError_t {
        cudaError_t a = cudaFuncSetAttribute(forward_tc_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_K1);
        if (a != cudaSuccess) return a;
        return cudaFuncSetAttribute(forward_tc_fused_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    });
    if (e != cudaSuccess) return e;
    FusedArgs fa;
    fa.q_mean = q_mean; fa.k_mean = k_mean; fa.index_out = index;
    fa.pool_cnt = sync; fa.route_flag = sync + d.B; fa.ctrl = ctrl;
    fa.units = d.R * (d.heads / 2);
    const int resident = tc_sm_count() * 4;
    // pooling runs this many images ahead of attention: the jobs of one wave of resident CTAs, plus the
    // time the routing of an image takes after its last unit is pooled
    int delta = (resident + fa.units - 1) / fa.units + 3;
    static const char* env = getenv("BRA_FUSED_DELTA");               // tuning aid
    if (env && atoi(env) > 0) delta = atoi(env);
    fa.delta = delta < d.B ? delta : d.B;
    fa.total = (d.B + fa.delta) * fa.units;
    fa.inject = inject;
    fa.sync_off = (int)(reinterpret_cast<char*>(sync) - reinterpret_cast<char*>(ctrl));
    fa.sync_bytes = (int)(sizeof(int32_t) * 2 * (size_t)d.B);
    const unsigned grid = (unsigned)(fa.total < resident ? fa.total : resident);
    e = launch_kernel(forward_tc_fused_kernel, dim3(grid), dim3(tc::THREADS), tc::SMEM_K1, st, false,
                      static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(K),
                      static_cast<const __nv_bfloat16*>(V), static_cast<const int32_t*>(index), lce_w, lce_b,
                      static_cast<__nv_bfloat16*>(O), lse, ctrl, d, 0, fa);
    count_launch();
    return e;
}

}  // namespace bra

