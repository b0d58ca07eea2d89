/*
 * vorta.h -- C ABI of the B200 (sm_100a) routed-attention library.
 *
 * The library computes the attention of one video-diffusion-transformer layer in
 * which every head is routed to one of three branches (VORTA, Section 3.3,
 * Eq. 4): full 3D attention (Section 2, Eq. 2), 3D sliding tile attention
 * (Section 3.2 and Appendix A.1, Algorithm 1), or core-set attention
 * unpool(attn(pool(.))) with bucketed core-set selection (Section 3.2;
 * Appendix A.1 "Bucketed coreset selection").
 *
 * Conventions shared by all entry points
 *   - Tokens are 0-based and frame-major: i = (t*H + h)*W + w, L = T*H*W.
 *   - Q, K, V, O are bf16, contiguous [B, heads, L, d]; d is 64 or 128.  With text tokens
 *     (vorta_plan_desc.text_tokens > 0) every "L" row count of a tensor argument below is
 *     L + text_tokens: the video tokens of a head, then its text tokens.
 *   - "dev" pointers are CUDA device memory, "host" pointers ordinary host
 *     memory.  The caller owns every buffer it passes and the stream; the library
 *     owns the plan and the small device tables inside it.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls enqueue work and return; argument errors are reported synchronously
 *     and launch nothing.
 *   - Every function returns a vorta_status; nothing throws, aborts or prints.
 *   - Device-side waits are bounded.  If one expires, the kernel records a code
 *     and leaves; vorta_device_status() reports it after the stream has drained.
 *   - A plan may be used from one thread at a time.
 */
#ifndef VORTA_H_
#define VORTA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define VORTA_API __attribute__((visibility("default")))
#else
#define VORTA_API
#endif

typedef struct vorta_plan vorta_plan; /* opaque */

typedef enum {
    VORTA_OK = 0,
    VORTA_ERR_INVALID_ARG = 1,  /* null pointer, size out of range, bad route id ... */
    VORTA_ERR_UNSUPPORTED = 2,  /* valid request this build cannot run (see vorta_plan_create) */
    VORTA_ERR_ALIGNMENT = 3,    /* a device pointer is not 16-byte aligned */
    VORTA_ERR_WORKSPACE = 4,    /* workspace missing or too small */
    VORTA_ERR_CUDA = 5,         /* a CUDA runtime/driver call failed */
    VORTA_ERR_TIMEOUT = 6,      /* a bounded device-side wait expired */
    VORTA_ERR_INTERNAL = 7      /* a self-check inside the library failed */
} vorta_status;

/* Branch ids, in the order of the gate vector [alpha_1, alpha_2, alpha_3] of
 * Section 3.3, Eq. 3: full, sliding-window, core-set. */
enum { VORTA_ROUTE_FULL = 0, VORTA_ROUTE_SLIDING = 1, VORTA_ROUTE_CORESET = 2 };

/* vorta_plan_desc.flags */
enum {
    VORTA_PLAN_HOST_ONLY = 1, /* geometry and accounting only: needs no GPU, cannot launch */
    VORTA_PLAN_POOL_MERGE = 2 /* core-set heads: the centre's rows of Q, K, V become the mean over the
                                 centre and the tokens pruned from its bucket before attending (Section 3.2
                                 mentions such a merge and does not give the operator).  With a
                                 bucket that keeps one token this is average pooling: bucket (2,1,1),
                                 (1,2,1) or (1,1,2) at ratio 0.5 are the AP variants of Section 4.2. */
};

/* Which attention kernel(s) vorta_routed_attention launches. */
enum {
    VORTA_KERNEL_TCGEN05 = 0, /* one persistent TMA + tcgen05/TMEM kernel, one CTA per SM, for every head */
    VORTA_KERNEL_SIMT = 1,    /* slow CUDA-core kernel over the same work lists (debug aid) */
    VORTA_KERNEL_PAIR = 2,    /* two launches: full and core-set heads in the CTA-pair kernel (cta_group::2
                                 MMAs, K/V shared by an SM pair), sliding heads in the TCGEN05 kernel after it.
                                 d = 128 and an even number of SMs; VORTA_ERR_UNSUPPORTED otherwise */
    VORTA_KERNEL_AUTO = 3     /* default: PAIR where it is supported and the full and core-set heads hold
                                 at least 60 % of the attention work of the call, else TCGEN05 */
};

typedef struct {
    int32_t B, heads;     /* batch, attention heads; >= 1 */
    int32_t T, H, W;      /* latent video grid (frames, height, width); T*H*W < 2^31 */
    int32_t d;            /* head dimension: 64 or 128 */
    int32_t tile[3];      /* sliding tile extent in tokens (tT, tH, tW) */
    int32_t window[3];    /* sliding window in TILES per axis (w_F, w_H, w_W of Algorithm 1), >= 1;
                             an even w acts like w + 1 (the test is |c - k| <= floor(w/2)) */
    int32_t bucket[3];    /* core-set bucket (t, h, w); {0,0,0} selects the paper's (2, 3, 2) */
    float coreset_ratio;  /* r_core in (0, 1]: a bucket of n tokens keeps max(1, floor(r*n + 1/2)) */
    float softmax_scale;  /* multiplies QK^T; 0 selects 1/sqrt(d) */
    const uint8_t *routes;/* host, [heads]: branch of each head (same for every batch entry) */
    int32_t flags;        /* bit set of VORTA_PLAN_* */
    int32_t device;       /* CUDA device ordinal; -1 = the calling thread's current device */
    int32_t text_tokens;  /* joint sequence of an MMDiT model: this many text tokens follow the T*H*W video
                             tokens in every head of Q, K, V, O (and X); 0 = video tokens only.  A text key
                             is visible to every query of every branch, a text query sees every key, and
                             core-set selection prunes video tokens only (every text token is kept).  The
                             paper runs HunyuanVideo (Section 4) without saying how its branches treat the
                             text tokens: this is this library's reading. */
} vorta_plan_desc;

typedef struct {
    int64_t L;                   /* video tokens per head (T*H*W); rows per head = L + text_tokens */
    int64_t Lc;                  /* core-set tokens per head (geometry only, data independent) */
    int32_t tiles_per_axis[3];   /* ceil(dim / tile) */
    int32_t n_tiles;
    int32_t n_buckets;
    int32_t kv_tiles_per_q_tile; /* prod_a min(tiles_a, 2*floor(w_a/2) + 1) */
    int32_t n_full, n_sliding, n_coreset; /* heads per branch under the current routes */
    int64_t workspace_bytes;     /* device workspace vorta_routed_attention needs (current routes) */
    int64_t workspace_bytes_max; /* ... if every head were routed to core-set */
    int64_t host_call_scratch_bytes; /* device scratch vorta_routed_attention_host needs */
    int64_t mixture_workspace_bytes; /* device workspace vorta_soft_mixture needs */
    /* Algorithmic work: 4*d*(query, key) pairs the method itself attends, per (batch, head). */
    double flops_full_head;      /* 4 d (L + Lt)^2, Lt = text_tokens */
    double flops_sliding_head;   /* 4 d * (sum over tile pairs in the window of valid tokens products
                                    + L Lt [video queries x text keys] + Lt (L + Lt) [text queries]) */
    double flops_coreset_head;   /* 4 d (Lc + Lt)^2 */
    double flops_layer;          /* B * sum over heads, current routes */
    double flops_issued_layer;   /* what the tensor cores are really given (padding to 128-row blocks
                                    and partial tiles included; not the idle half of the pair kernel's
                                    MMAs on a one-tile item); 0 for a host-only plan */
    int64_t n_work_items;        /* (head, query block) items of a call's attention stage; 0 for a host-only plan */
    /* Algorithmic bytes of the memory-bound stages, per core-set (batch, head). */
    int64_t select_bytes_head;   /* L*dx*2 read + (Lc + L)*4 written, with dx = d */
    int64_t gather_bytes_head;   /* 3 * (Lc + Lt)*d*2 read and written */
    int64_t scatter_bytes_head;  /* (Lc + Lt)*d*2 read + (L + Lt)*d*2 written */
    int64_t text_tokens;         /* Lt of the plan (0 = video tokens only) */
} vorta_plan_info_t;

/*
 * Build a plan for one layer shape: tile grid, window, buckets, core-set offsets,
 * the block-sparse sliding-tile mask (Algorithm 1, evaluated between tiles by a
 * CUDA kernel) and the ordered work list of the persistent attention kernel.
 * Reads desc and desc->routes (host) during the call only.  *out receives the
 * plan; free it with vorta_plan_destroy.
 * Unsupported (VORTA_ERR_UNSUPPORTED): d not in {64,128}; a tile that cannot be cut
 * into at most 8 equal boxes of at most 128 tokens (cuts along any of its axes; a
 * 6 x 9 x 8 tile is four 3 x 9 x 4 boxes, a tile of more than 1 024 tokens or a
 * 131-token one has no such cut); a tile extent > 256; a bucket with more than 32
 * tokens.
 */
VORTA_API int vorta_plan_create(const vorta_plan_desc *desc, vorta_plan **out);

/* Replace the per-head routes (Section 3.3: the router decides per diffusion
 * timestep); geometry tables are kept.  routes_host is [n] with n == heads.
 * Does not wait for the device: the plan keeps the work lists of the last four route
 * vectors, each in device buffers of its own.  A vector it still holds becomes current
 * at once (microseconds, nothing touches the device); a new one is built on the host
 * (about a millisecond for ten thousand work items) into the entry used least recently,
 * after a wait for the last call that ran THAT entry only, and copied up on a stream of
 * the plan.  Calls already enqueued keep the lists they were enqueued with.  If a rebuild
 * fails (VORTA_ERR_CUDA) the plan launches nothing (VORTA_ERR_INTERNAL) until a later
 * vorta_plan_set_routes succeeds. */
VORTA_API int vorta_plan_set_routes(vorta_plan *plan, const uint8_t *routes_host, int32_t n);

VORTA_API int vorta_plan_destroy(vorta_plan *plan);

VORTA_API int vorta_plan_info(const vorta_plan *plan, vorta_plan_info_t *out);

/*
 * Head-sharded multi-GPU use (heads are independent units: no exchange inside the
 * op): split the heads of the current routes over n_ranks devices so that the most
 * loaded rank is as light as longest-processing-time-first packing makes it.  The
 * cost of a head is its attention work under its route (flops_full_head,
 * flops_sliding_head or flops_coreset_head of vorta_plan_info).  Heads are taken in
 * descending cost (ties: ascending head index) and each goes to the rank with the
 * least work so far (ties: lowest rank).  Host arrays:
 *   rank_of_head   out, [heads]: rank in [0, n_ranks) of every head
 *   rank_flops     out, [n_ranks] or NULL: attention FLOPs per batch entry of each rank
 * Works on host-only plans.  The paper runs on one GPU; this is the partition a
 * caller with head-sharded Q, K, V (e.g. after an all-to-all upstream) needs, each
 * rank then creating a plan over its own heads.
 */
VORTA_API int vorta_shard_heads(const vorta_plan *plan, int32_t n_ranks, int32_t *rank_of_head,
                                double *rank_flops);

/*
 * Copy the canonical block mask to host memory: out_host is uint8
 * [n_tiles * n_tiles], BM[qt*n_tiles + kt] = 1 iff key tile kt lies in the window
 * of query tile qt (Algorithm 1 applied to tile ids, the query tile first moved
 * to its window-centre tile), with tile id = (tile_T*nt_H + tile_H)*nt_W + tile_W.
 * Not available on a host-only plan.
 */
VORTA_API int vorta_plan_block_mask(const vorta_plan *plan, uint8_t *out_host);

/* Select the attention kernel (VORTA_KERNEL_*).  Default VORTA_KERNEL_AUTO. */
VORTA_API int vorta_plan_set_kernel(vorta_plan *plan, int32_t kernel);

/* The kernel vorta_routed_attention uses with the current routes and selection: what
 * VORTA_KERNEL_AUTO resolves to, else the selected one.  Negative on a null or host-only plan. */
VORTA_API int32_t vorta_plan_kernel_in_use(const vorta_plan *plan);

/*
 * Bucketed core-set selection (Section 3.2; Appendix A.1): for every (b, hx)
 * slice of X and every bucket, score each token by its cosine similarity to the
 * bucket's centre token, prune the n - keep(n) most similar (ties: lower local
 * index first), keep the rest.
 *   X_dev        bf16 [B, Hx, L, dx], dx a multiple of 8, Hx >= 1
 *   core_idx_dev int32 [B, Hx, Lc] out: kept token ids, buckets in raster order, in
 *                each bucket the centre first, then the other kept tokens ascending
 *   src_slot_dev int32 [B, Hx, L]  out: position in core_idx of the token whose
 *                attention output each token receives (its own, or its centre's)
 * Precision of the scores: features of a width other than 128 are scored in fp64 (the
 * products of bf16 values are exact there).  For dx == 128 the scores are first taken in
 * fp32; a bucket in which two scores on either side of the keep/prune boundary lie within
 * 2^-13 of each other, or whose norms leave the range fp32 handles safely, is scored again
 * in fp64, so the decisions are the fp64 ones in both cases.
 */
VORTA_API int vorta_coreset_select(const vorta_plan *plan, const void *X_dev, int32_t Hx, int32_t dx,
                                   int32_t *core_idx_dev, int32_t *src_slot_dev, void *stream);

/*
 * One layer of routed attention: O[b, h] = branch_{routes[h]}(Q[b, h], K[b, h], V[b, h]).
 * Core-set heads: select on X (NULL = on K of that head; else bf16
 * [B, Hx, L, d] with Hx == 1, shared by all heads, or Hx == heads), gather the
 * kept rows of Q, K, V, attend, scatter back (Section 3.2, last paragraph).
 * Sliding heads: Algorithm 1's mask, only the listed tile pairs are computed.
 *   Q, K, V      device bf16 [B, heads, L + text_tokens, d], 16-byte aligned (per head: the
 *                L = T*H*W video tokens, then the text tokens)
 *   O            same shape, out; every element is written
 *   workspace    device, >= vorta_plan_info().workspace_bytes, 256-byte aligned
 *                (may be NULL when no head is routed to core-set); contents are
 *                scratch and undefined afterwards
 * Hx is the head count of X (ignored when X is NULL).
 * Launch order on `stream`: select, gather, attention, scatter.
 * Calls into this library on one device must be ordered with respect to each other (one
 * stream, or streams chained by events): the attention stage is made of persistent kernels
 * that each expect the whole GPU, and two of them from different calls running side by side
 * have been seen to starve each other until a bounded wait gave up (the call then reports
 * VORTA_ERR_TIMEOUT through vorta_device_status and O is incomplete).
 */
VORTA_API int vorta_routed_attention(const vorta_plan *plan, const void *Q, const void *K,
                                     const void *V, void *O, const void *X_or_null, int32_t Hx,
                                     void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same layer with HOST buffers (bf16 [B, heads, L, d]; pinned memory, or the
 * copies neither overlap nor return early).  The heads are worked through in up to
 * twelve groups, most expensive first: the plan's own copy-in stream brings a group's
 * Q, K, V into dev_scratch, the layer's kernels for that group run on `stream` or on
 * a second kernel stream of the plan (groups alternate, so that one group's kernels
 * start in the SMs the previous group's last blocks leave), and the plan's copy-out
 * stream returns its O, so that copies and kernels of different groups overlap.  The call starts after the work already enqueued on `stream` and
 * `stream` ends up waiting for the last copy out: to the caller it is one operation
 * on `stream`.  Returns after enqueueing (synchronise `stream` before reading
 * O_host or reusing dev_scratch from another stream).  The result is the one
 * vorta_routed_attention gives (bit for bit under a fixed kernel choice; under
 * VORTA_KERNEL_AUTO every group of heads makes its own choice, and a head served by
 * another kernel than in the one-call path may differ in the last bf16 bit).  dev_scratch: device memory of at least
 * vorta_plan_info().host_call_scratch_bytes, 256-byte aligned.  Two calls on the
 * same plan must not be in flight on different streams at once (they share the
 * plan's copy streams and events).  The first call after plan creation or a route
 * change builds the groups' work lists before it enqueues (small device allocations and
 * copies, after a wait for the previous host-buffer call of the plan).
 */
VORTA_API int vorta_routed_attention_host(const vorta_plan *plan, const void *Q_host,
                                          const void *K_host, const void *V_host, void *O_host,
                                          void *dev_scratch, size_t dev_scratch_bytes, void *stream);

/*
 * Router (Section 3.3, Eq. 3-4).  gates[h] = softmax(T . W_R[h]) and the branch the
 * inference rule selects for head h: sliding if its gate is strictly larger than the
 * other two, core-set likewise, full otherwise (every tie goes to full attention).
 *   T_dev      f32 [d_model]           timestep embedding
 *   WR_dev     f32 [heads, d_model, 3] router weights, gate order (full, sliding, core-set)
 *   gates_dev  f32 [heads, 3] out      routes_dev  uint8 [heads] out (device; copy to the
 *                                      host and pass to vorta_plan_set_routes)
 * Logits are accumulated in fp64; the rule is evaluated on the logits, which order
 * exactly like the gates.
 */
VORTA_API int vorta_router_gates(const float *T_dev, const float *WR_dev, int32_t d_model, int32_t heads,
                                 float *gates_dev, uint8_t *routes_dev, void *stream);

/*
 * Soft mixture of the three branches (Section 3.3, Eq. 5: the forward pass used to
 * train the router): O[b, h] = g[h][0] full(.) + g[h][1] sliding(.) + g[h][2] coreset(.).
 * Every head runs all three branches in one attention stage (one launch, or the two of
 * VORTA_KERNEL_PAIR; the plan's routes are ignored), then the branch outputs are combined in fp32.
 *   gates_dev  f32 [heads, 3], device
 *   workspace  device, >= vorta_plan_info().mixture_workspace_bytes, 256-byte aligned
 * Core-set selection is on K of each head.  The first call builds the work list
 * (synchronous copies to the device).
 */
VORTA_API int vorta_soft_mixture(vorta_plan *plan, const void *Q, const void *K, const void *V,
                                 const float *gates_dev, void *O, void *workspace, size_t workspace_bytes,
                                 void *stream);

/*
 * The same layer for callers that cannot allocate device memory -- code running
 * inside another framework's memory pool with no spare capacity, plug-ins that are
 * handed fixed tensors and forbidden to call cudaMalloc, services with a frozen
 * memory budget.  (The paper has no counterpart: this is an interface convenience.)
 * It behaves like vorta_routed_attention, but the core-set branch's scratch is a
 * fixed array inside the library of VORTA_STATIC_WORKSPACE_BYTES bytes, which every
 * GPU that loads the library holds until the process exits.
 *   - Plans whose vorta_plan_info().workspace_bytes exceeds that size are refused
 *     with VORTA_ERR_WORKSPACE and nothing is launched.
 *   - The call itself allocates nothing (no cudaMalloc/cudaFree, no allocating
 *     library routine).  The first call on each device looks up the array's device
 *     address (cudaGetSymbolAddress with that device current); make that first call
 *     before starting any stream capture.  With CUDA's lazy module loading that look-up
 *     is also the moment the driver sets the array's bytes aside on that device: on a
 *     device with no room left it fails, the call returns VORTA_ERR_CUDA and launches
 *     nothing.
 *   - All calls on a device share the one array.  It keeps whatever the last call
 *     left in it; nothing in it needs clearing, because every region is written
 *     before it is read within a call.  Two calls whose kernels overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them.
 * Q, K, V, O, X_or_null, Hx and stream are as for vorta_routed_attention.
 */
#define VORTA_STATIC_WORKSPACE_BYTES (16u * 1024u * 1024u)
VORTA_API int vorta_routed_attention_static(const vorta_plan *plan, const void *Q, const void *K,
                                            const void *V, void *O, const void *X_or_null, int32_t Hx,
                                            void *stream);

/* CUDA device ordinal the plan's tables live on (-1 for a host-only plan). */
VORTA_API int vorta_plan_device(const vorta_plan *plan, int32_t *device);

/*
 * Stage timing.  With profiling on, vorta_routed_attention records CUDA events
 * on its stream around its four stages.  After the stream has been synchronised,
 * vorta_plan_stage_ms returns the last call's durations in milliseconds:
 * ms[0] select, ms[1] gather, ms[2] attention, ms[3] scatter (0 if a stage did not run).
 */
VORTA_API int vorta_plan_set_profiling(vorta_plan *plan, int32_t on);
VORTA_API int vorta_plan_stage_ms(const vorta_plan *plan, float ms[4]);
/* The same for an earlier call: calls_back = 0 is the last profiled call, 1 the one
 * before it, ... up to 63.  VORTA_ERR_INVALID_ARG if that call was never made. */
VORTA_API int vorta_plan_stage_ms_at(const vorta_plan *plan, int32_t calls_back, float ms[4]);
/* The attention stage of that call by launch: ms[0] the first attention kernel (the pair kernel
 * under VORTA_KERNEL_PAIR, else the only one), ms[1] the single-CTA kernel that follows the pair
 * kernel for the sliding heads (0 if there was one launch). */
VORTA_API int vorta_plan_attention_ms_at(const vorta_plan *plan, int32_t calls_back, float ms[2]);

/* Number of kernels the last vorta_routed_attention call launched. */
VORTA_API int vorta_plan_last_launches(const vorta_plan *plan, int32_t *n);

/*
 * Synchronise `stream` and report whether a kernel of this plan gave up on a
 * bounded wait: *code_out = 0 if none did, else a non-zero location code.
 * Returns VORTA_ERR_TIMEOUT in that case and clears the code.
 */
VORTA_API int vorta_device_status(const vorta_plan *plan, void *stream, int32_t *code_out);

VORTA_API const char *vorta_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* VORTA_H_ */
