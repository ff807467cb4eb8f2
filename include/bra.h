/*
 * bra.h - C boundary of the B200 (sm_100a) Bi-Level Routing Attention library.
 *
 * The library computes the hot path of BRA (BiFormer, arXiv 2303.08810,
 * Section 3.2, Algorithm 1) starting from already-projected Q, K, V:
 *   1. region mean pooling of Q and K            (Section 3.2, "per-region average")
 *   2. region affinity A^r = Q^r (K^r)^T         (Eq. 4)
 *   3. row-wise top-k routing index I^r          (Eq. 5)
 *   4. token-to-token softmax attention over the keys/values of the k routed
 *      regions, K^g / V^g never written to memory (Eq. 6, Eq. 7 with Eq. 1)
 *   5. + LCE(V), a 5x5 depthwise convolution of V (Eq. 7)
 * and the gradients of step 4-5 for a fixed routing index.
 *
 * Common rules for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte
 *     aligned, dense and contiguous.  The library allocates no device memory
 *     and keeps no state between calls besides kernel attributes and launch
 *     choices remembered per device and problem shape, and one helper stream
 *     with two events per device and host thread (created by the first
 *     bra_backward call; its work is forked from and joined back into `stream`).
 *   - Q, K, V, O, dO, dQ, dK, dV: [B, H, W, C], element type p->dtype, channel
 *     c = head * (C / heads) + j (concat order of Eq. 2).
 *   - Regions: S x S non-overlapping blocks of (H/S) x (W/S) tokens, numbered
 *     row-major r = ry * S + rx (region partition, Section 3.2).  Where S does
 *     not divide H or W (Appendix C picks S as a divisor "to avoid padding"),
 *     the library works on copies of Q, K, V zero-padded at the bottom and the
 *     right to the next multiples of S: the zero tokens are pooled, routed to
 *     and attended to like real ones, and O, lse and the gradients are cropped
 *     back to H x W.  The copies live in ws (bra_workspace_bytes accounts for
 *     them) and cost one extra kernel per tensor.
 *   - index: int32 [B, heads, S*S, topk] (or [B, 1, S*S, topk] when
 *     p->shared_routing != 0).  Row i lists the key regions that the queries of
 *     region i attend to.  It is a list: any order, duplicates count twice.
 *   - ws: scratch of at least bra_workspace_bytes(p) bytes, 256-byte aligned.
 *     It holds a device status block (error words and, for the one-launch
 *     forward, barrier counters) that the kernels expect to find ZERO and
 *     leave zero: before its first use fill ws with zeros or call
 *     bra_workspace_init().  bra_device_status() restores that state when it
 *     reports an error.  Calls that share a ws must be ordered on one stream.
 *   - Every call is asynchronous on `stream` (a cudaStream_t passed as void*).
 *   - Errors a host check can find return synchronously, nothing launched,
 *     outputs untouched.  Errors only the device can see (an out-of-range
 *     entry in a caller's index) never trap: the offending work is skipped,
 *     a code is recorded in ws and bra_device_status() reports it.
 *   - Outputs must not alias inputs.
 */
#ifndef BRA_H_
#define BRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum bra_status {
    BRA_OK = 0,
    BRA_ERR_NULL = 1,        /* a required pointer is NULL */
    BRA_ERR_SHAPE = 2,       /* B,H,W,C,heads,S <= 0; heads does not divide C */
    BRA_ERR_TOPK = 3,        /* topk < 1 or topk > S*S */
    BRA_ERR_DTYPE = 4,       /* dtype is not BRA_F32 / BRA_BF16 */
    BRA_ERR_ALIGN = 5,       /* a pointer is not 16-byte aligned (ws: 256) */
    BRA_ERR_WORKSPACE = 6,   /* ws_bytes < bra_workspace_bytes(p) */
    BRA_ERR_UNSUPPORTED = 7, /* valid problem this build has no kernel for (head dim, lce_ksize, impl) */
    BRA_ERR_CUDA = 8,        /* a CUDA runtime call failed (launch, attribute) */
    BRA_ERR_INDEX = 9,       /* device-detected: routing index entry outside [0, S*S) */
    BRA_ERR_TIMEOUT = 10,    /* device-detected: a bounded wait gave up */
    BRA_ERR_STATIC_LIMIT = 11 /* bra_route_static only: B*S*S*C > BRA_ROUTE_STATIC_MAX_MEAN_FLOATS */
} bra_status;

typedef enum bra_dtype { BRA_F32 = 0, BRA_BF16 = 1 } bra_dtype;

/* Which kernel family runs the token-to-token attention (step 4-5). */
typedef enum bra_impl {
    BRA_IMPL_AUTO = 0,  /* fastest kernel that supports the problem */
    BRA_IMPL_SIMT = 1,  /* fp32 CUDA-core kernel: any dtype, any shape with C/heads <= 128 */
    BRA_IMPL_MMA = 2,   /* bf16 warp-level tensor-core kernel (C/heads == 32) */
    BRA_IMPL_TC = 3,    /* bf16 tcgen05/TMEM kernels (C/heads == 32; regions of 8 x 8 tokens, or 16 wide and a multiple of 8 high) */
    BRA_IMPL_IMG = 4,   /* bf16 warp-level tensor-core kernel with a whole (image, head) of K and V resident in
                           shared memory (C/heads == 32, H*W <= ~1500 tokens): small maps, small regions */
    BRA_IMPL_TC_FUSED = 5 /* as BRA_IMPL_TC, and bra_forward runs pooling, routing and attention as three phases of
                           ONE launch (8 x 8-token regions, topk = 1, per-head routing, <= 64 regions,
                           C <= 128): results equal to the chain of launches bit for bit */
} bra_impl;

/*
 * Failure injection for tests of the error path (no GPU fault, trap or hang is involved).
 * BRA_INJECT_LOSE_POOLED_UNIT: in the one-launch forward (bra_forward with BRA_IMPL_TC_FUSED) one pooled
 * unit is never counted as done, so every CTA's bounded wait for the end of the pooling phase runs out
 * after a few thousand polls, before any tensor-core work or tile copy has been issued;
 * the kernel returns normally, O is not written and bra_device_status() reports BRA_ERR_TIMEOUT.
 * Ignored by every other path.
 */
typedef enum bra_inject { BRA_INJECT_NONE = 0, BRA_INJECT_LOSE_POOLED_UNIT = 1 } bra_inject;

/* Problem statement in the notation of Algorithm 1 (H, W, C, S, k) plus batch and heads. */
typedef struct bra_problem {
    int32_t B, H, W, C;     /* batch, feature-map height and width, channels */
    int32_t heads;          /* attention heads; head dim d = C / heads (Eq. 2) */
    int32_t S;              /* regions per side: S x S regions */
    int32_t topk;           /* k of Eq. 5, 1 <= k <= S*S */
    int32_t dtype;          /* bra_dtype of Q, K, V, O and their gradients */
    float   scale;          /* softmax scale of Eq. 1; <= 0 selects 1/sqrt(C/heads) */
    int32_t shared_routing; /* 0: one index per head (affinity over the head's channels);
                               1: one index for all heads (Eq. 4 read over all C channels) */
    int32_t lce_ksize;      /* 5: add LCE(V) (Eq. 7); 0: attention term only */
    int32_t impl;           /* bra_impl */
    int32_t inject;         /* bra_inject: 0 in production */
} bra_problem;

/* Scratch size in bytes every call on problem p needs (0 if p is invalid). Host only. */
size_t bra_workspace_bytes(const bra_problem* p);

/*
 * Puts ws into the state the kernels expect: status block (error words, barrier counters) zero
 * (an asynchronous memset on `stream`; the rest of ws needs no initial value).  Needed once before the
 * first use of a ws that was not zero-filled.  (Housekeeping of this library: Algorithm 1 has no
 * counterpart.)
 */
bra_status bra_workspace_init(const bra_problem* p, void* ws, size_t ws_bytes, void* stream);

/*
 * Region-to-region routing (Section 3.2: per-region average; Eq. 4; Eq. 5).
 *   Q, K     in   [B,H,W,C]
 *   q_mean   out  fp32 [B, S*S, C], Q^r; may be NULL (kept in ws only)
 *   k_mean   out  fp32 [B, S*S, C], K^r; may be NULL
 *   index    out  int32 [B, heads|1, S*S, topk]; row order: affinity descending,
 *                 equal affinities by ascending region number
 * Means are accumulated and the affinity evaluated in fp32 whatever the dtype.
 */
bra_status bra_route(const bra_problem* p, const void* Q, const void* K,
                     float* q_mean, float* k_mean, int32_t* index,
                     void* ws, size_t ws_bytes, void* stream);

/*
 * bra_route for callers that cannot hand over scratch memory.  (The paper has
 * no counterpart: this is a packaging variant of bra_route, same arithmetic.)
 *
 * Who needs it: code that runs where device memory must not be allocated or
 * sized at call time - a plug-in inside a host application that owns the
 * memory pool and forbids cudaMalloc, a real-time loop where an allocation's
 * implicit synchronisation is not acceptable, or a caller that simply has no
 * allocator to ask for a `ws` buffer.  bra_route needs `ws` (or caller
 * buffers) for the region means Q^r, K^r between its pooling and its routing
 * kernel; here those means live in a fixed array inside the library image.
 *
 *   Q, K     in   [B,H,W,C] device pointers, as for bra_route
 *   index    out  int32 [B, heads|1, S*S, topk], as for bra_route (bit-identical result)
 *
 * Limits and rules
 *   - B * S*S * C must not exceed BRA_ROUTE_STATIC_MAX_MEAN_FLOATS, otherwise
 *     BRA_ERR_STATIC_LIMIT is returned and nothing is launched.  The array
 *     (2 x that many floats = 4 MiB) is part of the library: every GPU that
 *     loads it carries the array until the process exits.
 *   - The call itself allocates nothing on host or device and frees nothing.
 *   - The first call on each device looks up the array's device address (a
 *     driver query, no allocation).  Make that first call outside any stream
 *     capture; later calls on that device only launch kernels.
 *   - All calls on a device share the one array.  Two calls whose kernels can
 *     overlap on the GPU (different streams, no dependency) race on it: order
 *     them.  The array keeps the previous call's means; nothing in it has to
 *     be zero, because pooling overwrites every element routing then reads.
 *   - The region means are not returned; use bra_route to get them.
 *   - S must divide H and W here (BRA_ERR_UNSUPPORTED otherwise): the padded
 *     copies of Q and K that bra_route makes for other maps would need scratch.
 */
#define BRA_ROUTE_STATIC_MAX_MEAN_FLOATS (512 * 1024)
bra_status bra_route_static(const bra_problem* p, const void* Q, const void* K,
                            int32_t* index, void* stream);

/*
 * Token-to-token attention over routed regions plus LCE (Eq. 6, Eq. 7, Eq. 1):
 *   O = softmax(scale * Q K^g^T) V^g + LCE(V).
 *   index    in   as above (the caller's or bra_route's)
 *   lce_w    in   fp32 [C,5,5]; out[y,x,c] += sum_ij w[c,i,j] V[y+i-2, x+j-2, c], zero outside
 *                 the map; NULL allowed iff p->lce_ksize == 0
 *   lce_b    in   fp32 [C] bias added with LCE; may be NULL
 *   O        out  [B,H,W,C]
 *   lse      out  fp32 [B, heads, H*W]: log of the softmax denominator (natural log, scaled
 *                 scores) of each query; may be NULL.  bra_backward needs it.
 */
bra_status bra_attend(const bra_problem* p, const void* Q, const void* K, const void* V,
                      const int32_t* index, const float* lce_w, const float* lce_b,
                      void* O, float* lse, void* ws, size_t ws_bytes, void* stream);

/*
 * Algorithm 1 from the projected Q, K, V on: bra_route then bra_attend in one call; same results,
 * bit for bit, as the two calls.  The library's kernels are chained on `stream` and overlap at their
 * ends; with BRA_IMPL_TC_FUSED the whole call is one kernel launch.
 *   index    out  may be NULL (then kept in ws only)
 *   lse      out  may be NULL
 */
bra_status bra_forward(const bra_problem* p, const void* Q, const void* K, const void* V,
                       const float* lce_w, const float* lce_b, void* O,
                       int32_t* index, float* lse, void* ws, size_t ws_bytes, void* stream);

/*
 * Gradients of Eq. 7 for a fixed routing index (top-k is not differentiable,
 * so nothing flows through pooling or Eq. 4).  With P the softmax of Eq. 1:
 *   dV^g = P^T dO, dP = dO V^g^T, dS = P o (dP - rowsum(P o dP)),
 *   dQ = scale dS K^g, dK^g = scale dS^T Q, rows of dK^g / dV^g added back to
 *   the regions they were gathered from; LCE: dV += corr^T(dO, w),
 *   d_lce_w[c,i,j] = sum_{b,y,x} dO[b,y,x,c] V[b,y+i-2,x+j-2,c], d_lce_b[c] = sum dO.
 *   lse      in   from bra_attend / bra_forward on the same inputs
 *   dQ,dK,dV out  [B,H,W,C], dtype of p
 *   d_lce_w  out  fp32 [C,5,5]; may be NULL iff p->lce_ksize == 0
 *   d_lce_b  out  fp32 [C]; may be NULL
 * The summation order is fixed: results are bit-identical from run to run.
 */
bra_status bra_backward(const bra_problem* p, const void* Q, const void* K, const void* V,
                        const int32_t* index, const float* lce_w, const float* lse,
                        const void* dO, void* dQ, void* dK, void* dV,
                        float* d_lce_w, float* d_lce_b,
                        void* ws, size_t ws_bytes, void* stream);

/*
 * Synchronises `stream`, then returns and clears the first device-detected
 * error recorded in ws (BRA_OK, BRA_ERR_INDEX, BRA_ERR_TIMEOUT, or BRA_ERR_CUDA
 * if the synchronisation itself failed).  When it reports an error it also puts the
 * barrier counters in ws back to zero (as bra_workspace_init does), so the next call
 * starts clean.  ws must have been initialised and used by an earlier call.
 */
bra_status bra_device_status(void* ws, void* stream);

/* Number of kernels launched by the last bra_* call on this thread (host-side count). */
int32_t bra_last_launch_count(void);

/* Static description of a status code. Never NULL. */
const char* bra_status_string(bra_status s);

/* Library version: major * 10000 + minor * 100 + patch. */
int32_t bra_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BRA_H_ */
