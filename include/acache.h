/*
 * acache.h -- C ABI of the affix-cache refresh path for bidirectional diffusion LLMs
 *             (ACache: anchor scoring, top-K anchor selection, selective
 *             recomputation, KV scatter), implemented as CUDA kernels for sm_100a.
 *
 * Notation (Section 3.1-3.3 of the paper): the shared affix is the contiguous span
 * F = {l .. r} of L positions inside a T-token context; M is the set of masked
 * generation positions (m = |M|); A is the Anchor set (K = |A|), S = F \ A; E is the
 * set of request-specific positions recomputed together with the anchors (e = |E|);
 * R = A u E is the recompute set.  The layer is the pre-norm RMSNorm / RoPE / SwiGLU
 * layer of LLaDA-8B and Dream-7B: D hidden, H query heads, Hkv KV heads, d head dim,
 * Fm MLP width.
 *
 * Conventions that hold for every entry point
 *  - Pointers marked DEVICE are device addresses on the current CUDA device; pointers
 *    marked HOST are host addresses.  All device pointers must be 16-byte aligned.
 *  - bf16 tensors are row-major with the last index contiguous.  Weights are
 *    [out, in].  The KV cache is token-major [B, ctx_capacity, Hkv, d]; K is stored
 *    after the rotary embedding.
 *  - Ownership: the caller owns every buffer (weights, cache, inputs, outputs and the
 *    workspace).  The library allocates only the small host-side context object in
 *    acache_create and frees only that in acache_destroy.
 *  - Asynchrony: every compute entry point only enqueues work on the given stream and
 *    returns; it never synchronises.  Calls that share one context must be issued on
 *    one stream (they share the workspace).
 *  - Weights are constants of a call: the kernels may start reading them (shared-memory
 *    ring prefill, L2 requests) before the work enqueued earlier on the stream has
 *    finished.  They must therefore be complete and visible before the call is enqueued;
 *    in particular they must not be written by the kernel that immediately precedes the
 *    call on the same stream (a weight copy or a dequantisation): put an event or any
 *    other kernel in between, or synchronise.  Every other input (x, the cache, index
 *    arrays, scores) follows plain stream order.
 *  - Errors: every call returns acache_status.  Argument and shape validation happens
 *    on the host before any launch, so a non-OK status means nothing was enqueued.
 *    Faults that depend on device data (an index outside its range) never trap: the
 *    offending row is skipped and a bit is set in a device status word that
 *    acache_poll_status reads back.
 *  - Compact row order: every "[B, K+e, ...]" tensor lists, per request, the K anchor
 *    rows in ascending position followed by the e extra rows in the order given.
 */
#ifndef ACACHE_H_
#define ACACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ACACHE_OK = 0,
    ACACHE_ERR_INVALID_ARG = 1,       /* NULL / misaligned pointer, negative size, bad range   */
    ACACHE_ERR_UNSUPPORTED_SHAPE = 2, /* shape outside what the kernels are built for          */
    ACACHE_ERR_WORKSPACE = 3,         /* workspace missing or smaller than acache_workspace_bytes */
    ACACHE_ERR_CUDA = 4,              /* a CUDA runtime call failed (see acache_last_error)    */
    ACACHE_ERR_TIMEOUT = 5            /* a bounded device-side wait expired (status word)      */
} acache_status;

/* bits of the device status word returned by acache_poll_status */
#define ACACHE_FLAG_BAD_INDEX   0x1u  /* an anchor / masked / extra index was out of range; row skipped */
#define ACACHE_FLAG_WAIT_EXPIRED 0x2u /* a bounded wait inside a kernel gave up                          */

/* flags of acache_layer_step */
#define ACACHE_F_SCORE            0x1u /* form Q for the masked rows from x and run the scoring (Eq. 4-5) */
#define ACACHE_F_SELECT           0x2u /* run the top-K selection (Eq. 6); otherwise use the given anchor_idx */
#define ACACHE_F_ACCUMULATE       0x4u /* scores += this layer's scores (Eq. 5 sums over layers)        */
#define ACACHE_F_SCORE_NORM_FULL  0x8u /* softmax of Eq. 4 over every key of the context, not the affix only */
#define ACACHE_F_NO_RECOMPUTE    0x10u /* stop after scoring / selection (the selection-time probe)     */
#define ACACHE_F_DROP_NON_ANCHOR 0x20u /* DropNA layout (Section 5.3): the non-anchor affix entries are discarded, i.e. the
                                          recomputed rows attend the anchors and the non-affix positions only            */

typedef struct CUstream_st *acache_stream_t;   /* a cudaStream_t */
typedef struct acache_ctx acache_ctx;           /* opaque */

/* Layer shape and the largest problem the context must hold (sizes the workspace). */
typedef struct {
    int32_t hidden, n_heads, n_kv_heads, head_dim, ffn;
    float   rms_eps;
    int32_t qkv_bias;      /* 0/1: bq, bk, bv present */
    int32_t max_batch;     /* B                                  */
    int32_t max_ctx;       /* T (and the cache's ctx_capacity)   */
    int32_t max_affix;     /* L                                  */
    int32_t max_rows;      /* K + e per request                  */
    int32_t max_masked;    /* m per request                      */
    int32_t max_vocab;     /* V of acache_predict_commit, 0 if unused          */
    int32_t max_block;     /* rows per request of acache_predict_commit, 0 if unused */
} acache_model_desc;

/* DEVICE bf16 weights, [out, in] row-major.  bq/bk/bv may be NULL when qkv_bias == 0. */
typedef struct {
    const void *attn_norm_g;          /* [D]            */
    const void *wq, *wk, *wv;         /* [H*d, D], [Hkv*d, D], [Hkv*d, D] */
    const void *bq, *bk, *bv;         /* [H*d], [Hkv*d], [Hkv*d]          */
    const void *wo;                   /* [D, H*d]       */
    const void *mlp_norm_g;           /* [D]            */
    const void *w_gate, *w_up;        /* [Fm, D]        */
    const void *w_down;               /* [D, Fm]        */
} acache_layer_weights;

/* One layer's KV cache: DEVICE bf16 [B, ctx_capacity, Hkv, d]; request b starts at
 * element offset b * batch_stride (normally ctx_capacity * Hkv * d).
 * batch_stride == 0: ONE cache [ctx_capacity, Hkv, d] shared by every request of the batch (the
 * shared-affix storage of Section 4.1).  Accepted by the calls that only read the cache:
 * acache_score_anchors, and acache_recompute_anchors, whose k_new / v_new are then the requests'
 * private slots (anchors + request rows) and whose attention reads every other position from
 * the shared copy.  Calls that write the cache reject it. */
typedef struct {
    void   *k, *v;
    int64_t batch_stride;
    int32_t ctx_capacity;
} acache_kv;

/* The request batch: every request shares the layout (ctx_len, affix span, m, e). */
typedef struct {
    int32_t batch, ctx_len;
    int32_t affix_start, affix_len;       /* F = [affix_start, affix_start + affix_len)          */
    const int32_t *masked_pos;            /* DEVICE [B, n_masked] absolute positions outside F   */
    int32_t n_masked;
    const int32_t *extra_rows;            /* DEVICE [B, n_extra] absolute positions outside F; may be NULL when n_extra == 0 */
    int32_t n_extra;
    const float *rope_cos, *rope_sin;     /* DEVICE fp32 [>= ctx_len, d/2] rotary table, pairing (i, i + d/2) */
    const int32_t *token_ids;             /* optional DEVICE [B, ctx_len]: when set, the non-compact `x` of a call is an
                                             embedding table bf16 [n_embed, D] and position t of request b reads row
                                             token_ids[b, t] (an id outside [0, n_embed) raises ACACHE_FLAG_BAD_INDEX) */
    int32_t n_embed;
} acache_request;

/* ---- context ------------------------------------------------------------------------ */

/* Creates the host-side context for one layer shape.  Validates the shape:
 * head_dim in {64, 128}; n_heads % n_kv_heads == 0; hidden, H*d, Hkv*d and ffn
 * multiples of 128.  No device memory is allocated. */
acache_status acache_create(const acache_model_desc *desc, acache_ctx **out);

/* Bytes of device scratch the context needs for the sizes in its descriptor. */
size_t acache_workspace_bytes(const acache_ctx *ctx);

/* Hands the context its scratch: DEVICE memory, 256-byte aligned, at least
 * acache_workspace_bytes.  The caller keeps ownership and must keep it alive while
 * the context is used.  Enqueues a memset of the status word on `stream`. */
acache_status acache_set_workspace(acache_ctx *ctx, void *dev_ptr, size_t bytes, acache_stream_t stream);

void acache_destroy(acache_ctx *ctx);

/* Text of the last error recorded by this context (HOST string owned by the context). */
const char *acache_last_error(const acache_ctx *ctx);

/* Copies the device status word to *host_flags (HOST), synchronising `stream`, and
 * clears it.  Returns ACACHE_ERR_TIMEOUT if ACACHE_FLAG_WAIT_EXPIRED is set. */
acache_status acache_poll_status(acache_ctx *ctx, acache_stream_t stream, uint32_t *host_flags);

/* Failure-detection self-test (the paper has no counterpart).  Every wait inside the kernels (mbarrier or
 * grid-wide barrier) is bounded; when one runs out the kernel stops issuing work, waits for its copies in
 * flight, frees its tensor memory, raises ACACHE_FLAG_WAIT_EXPIRED and returns, and the context stays usable.
 * This call makes that happen once, on purpose: the next Q/K/V projection this context launches
 * (acache_recompute_anchors, acache_layer_step, ...) gives the grid-wide barrier that ends its row-preparation
 * phase a target one arrival beyond what its grid can deliver and a short poll limit (about a millisecond),
 * so the wait runs out before any tensor-core work was issued.  The call that contains it still enqueues its
 * later kernels, whose outputs are then meaningless; acache_poll_status afterwards returns ACACHE_ERR_TIMEOUT
 * and re-arms the barrier, and the next call on the context runs normally.  Nothing faults, traps or spins
 * without a bound. */
acache_status acache_debug_expire_next_wait(acache_ctx *ctx);

/* Number of kernels this context has launched since creation (for accounting). */
uint64_t acache_launch_count(const acache_ctx *ctx);

/* Measurement aid (the paper has no counterpart).  The stages of acache_layer_step, in
 * launch order; a stage's time runs from its first launch to the next stage's. */
enum {
    ACACHE_STAGE_MASK_Q = 0,    /* RMSNorm + Q projection + RoPE of the masked rows  */
    ACACHE_STAGE_SCORE,         /* Eq. 4-5                                            */
    ACACHE_STAGE_TOPK,          /* Eq. 6                                              */
    ACACHE_STAGE_GATHER_NORM,   /* row plan of R, gather, RMSNorm                     */
    ACACHE_STAGE_QKV,           /* QKV projection + RoPE + KV scatter                 */
    ACACHE_STAGE_ATTENTION,     /* attention of R over the whole context              */
    ACACHE_STAGE_OPROJ,         /* output projection + residual                       */
    ACACHE_STAGE_MLP_NORM,      /* second RMSNorm                                     */
    ACACHE_STAGE_GATE_UP,       /* gate/up projection + SwiGLU                        */
    ACACHE_STAGE_DOWN,          /* down projection + residual                         */
    ACACHE_N_STAGES
};

/* enable != 0: every following acache_layer_step records a CUDA event on its stream
 * before each stage (the first call creates the events; they serialise the stages, so a
 * timed step is slightly slower than an untimed one).  enable == 0 switches it off. */
acache_status acache_stage_timing(acache_ctx *ctx, int enable);

/* Waits for the last timed acache_layer_step and writes the milliseconds each stage took
 * to ms[ACACHE_N_STAGES] (HOST); stages that did not run read 0. */
acache_status acache_read_stage_times(acache_ctx *ctx, float *ms);

/* ---- the path ------------------------------------------------------------------------ */

/* Eq. 4-5 (Section 3.2), one layer's term:
 *   a[j,k,h] = Softmax_j( q_mask[k,h,:] . K_affix[j,kv(h),:] / sqrt(d) ),  j in F
 *   scores[b,j] (+)= sum_h sum_{k in M} a[j,k,h]
 * q_mask: DEVICE bf16 [B, m, H, d], the post-RoPE queries of the masked positions.
 * kv: the layer's cache; the affix keys are rows affix_start.. of each request.
 * scores: DEVICE fp32 [B, L].  accumulate != 0 adds to the existing contents.
 * norm_full != 0 takes the softmax over all ctx_len keys and keeps the affix columns.
 * The sum over heads and queries is evaluated in a fixed order (bitwise reproducible). */
acache_status acache_score_anchors(acache_ctx *ctx, const acache_request *req, const void *q_mask,
                                   const acache_kv *kv, float *scores, int accumulate, int norm_full,
                                   acache_stream_t stream);

/* The same scoring for callers that cannot allocate device memory (the paper has no
 * counterpart).  Some hosts of this library may not call cudaMalloc at all: code running
 * inside a CUDA-graph capture or a real-time loop, plug-ins handed a fixed memory budget by
 * their framework, or processes whose allocator is owned by someone else -- so they cannot
 * provide the workspace acache_score_anchors needs either.  This variant takes no context
 * and no workspace: its scratch is a 4 MiB array built into the library's device image
 * (every GPU that loads the library holds it until the process exits).
 *   shape: only n_heads, n_kv_heads and head_dim are read.
 *   Limit: B * H * (2 * m * ceil(keys / 256) + L) floats must fit in 2^20 floats, where keys
 *   is L (or ctx_len with norm_full); larger problems return ACACHE_ERR_WORKSPACE and
 *   enqueue nothing.  m <= 4096.
 * The first call on each device looks up the array's device address (with that device
 * current) and keeps it for the life of the process; make that first call before any stream
 * capture, and do not call cudaDeviceReset between calls (the kept address would be stale).
 * It calls no cudaMalloc, cudaFree or other allocating routine.  All calls share the one
 * array, which keeps the previous call's contents (nothing in it needs clearing: each call
 * overwrites what it reads), so two calls whose kernels may overlap on the GPU (different
 * streams) race; issue them on one stream or order them with events.
 * Inputs (kv->batch_stride = 0 included), outputs and results are those of
 * acache_score_anchors up to the order of fp32 additions: with no context there is no status
 * word for a bounded wait to report to, so this variant always runs the mma.sync scoring
 * kernels, also at the sizes where acache_score_anchors switches to its tcgen05 kernels
 * (about twice as fast at 8192 keys). */
acache_status acache_score_anchors_static(const acache_model_desc *shape, const acache_request *req,
                                          const void *q_mask, const acache_kv *kv, float *scores,
                                          int accumulate, int norm_full, acache_stream_t stream);

/* K of Eq. 6 from the recompute ratio: ceil(ratio * L) clipped to [0, L].  HOST, pure. */
int32_t acache_k_from_ratio(int32_t affix_len, double ratio);

/* Eq. 6 (Section 3.2): A = TopK({s_j}, K).  scores: DEVICE fp32 [B, L].
 * anchor_idx: DEVICE int32 [B, K], positions relative to affix_start, ascending.
 * Ties are broken towards the lower position, so the result is unique. */
acache_status acache_select_topk(acache_ctx *ctx, const float *scores, int32_t batch, int32_t affix_len,
                                 int32_t k, int32_t *anchor_idx, acache_stream_t stream);

/* The KV-deviation selector the paper compares its own against (appendix "CacheBlend-Style Anchor
 * Selection"): affix token j is ranked by how far its cached K/V (kv_ref: the affix-only / stale cache)
 * lie from its K/V under the full prompt (kv_full), without looking at the masked positions:
 *   scores[b,j] (+)= sum_{h,c} (K_full[b,l+j,h,c] - K_ref[b,l+j,h,c])^2 + (V_full[...] - V_ref[...])^2
 * (squared Euclidean distance over K and V together; the paper does not fix the norm).  One call is one
 * layer's term; accumulate != 0 adds to scores, so that the layers sum as in Eq. 5, and
 * acache_select_topk then picks the anchors exactly as for the attention scores.
 * kv_ref, kv_full: layout as acache_kv; either may have batch_stride 0 (one copy for the batch).  Only the
 * affix rows are read.  scores: DEVICE fp32 [B, L].  The sum is evaluated in a fixed order. */
acache_status acache_score_kv_deviation(acache_ctx *ctx, const acache_request *req, const acache_kv *kv_ref,
                                        const acache_kv *kv_full, float *scores, int accumulate,
                                        acache_stream_t stream);

/* Selective recomputation (Section 3.3, Section 4.3) of the rows R = A u E of every
 * request, WITHOUT touching the cache:
 *   xn = RMSNorm(x_r) g1; q,k,v = W{q,k,v} xn (+b); RoPE(q,k; position r)
 *   o  = bidirectional attention of q over all ctx_len keys/values, where positions in
 *        R read the fresh k/v and all others read the cache (store-then-attend view)
 *   y  = h1 + Wd (silu(Wg xn2) * (Wu xn2)),  h1 = x_r + Wo o,  xn2 = RMSNorm(h1) g2
 * x: DEVICE bf16, [B, ctx_len, D] (rows gathered by position) or, if x_is_compact,
 *    [B, K+e, D] in compact row order.
 * anchor_idx: DEVICE int32 [B, K] (relative to affix_start); k may be 0.
 * k_new, v_new: DEVICE bf16 [B, K+e, Hkv, d] out.  y: DEVICE bf16 [B, K+e, D] out. */
acache_status acache_recompute_anchors(acache_ctx *ctx, const acache_layer_weights *w,
                                       const acache_request *req, const acache_kv *kv,
                                       const void *x, int x_is_compact,
                                       const int32_t *anchor_idx, int32_t k,
                                       void *k_new, void *v_new, void *y, acache_stream_t stream);

/* Working-cache construction (Section 3.3, Section 4.1): writes the fresh K/V of the
 * rows R into the cache rows they belong to; every other row is left untouched
 * (byte-identical).  k_new/v_new as produced by acache_recompute_anchors. */
acache_status acache_scatter_kv(acache_ctx *ctx, const acache_request *req, acache_kv *kv,
                                const int32_t *anchor_idx, int32_t k,
                                const void *k_new, const void *v_new, acache_stream_t stream);

/* One layer-step on one stream: [score -> select ->] recompute -> scatter, with the
 * scatter fused into the QKV projection and attention reading the updated cache
 * (store-then-attend, Appendix C.1).  Gives the same cache and (within rounding of
 * the attention tiling) the same y as the three split calls in sequence.
 *   flags & ACACHE_F_SCORE : scores is written.  With a compact x the masked positions must be
 *                            among extra_rows (their rows are looked up there); a masked position
 *                            that is not raises ACACHE_FLAG_BAD_INDEX.
 *   flags & ACACHE_F_SELECT: anchor_idx [B, K] is written, K = acache_k_from_ratio(L, ratio);
 *                            otherwise anchor_idx is an input with that K.
 *   flags & ACACHE_F_DROP_NON_ANCHOR: the DropNA ablation of Section 5.3: K/V of R are refreshed and
 *                            written as usual, but the attention of the rows of R skips every affix position
 *                            that is not an anchor (accepted by acache_layer_step_shared as well).
 * scores: DEVICE fp32 [B, L] (may be NULL without F_SCORE/F_SELECT).
 * y: DEVICE bf16 [B, K+e, D]. */
acache_status acache_layer_step(acache_ctx *ctx, const acache_layer_weights *w,
                                const acache_request *req, acache_kv *kv,
                                const void *x, int x_is_compact, double ratio, uint32_t flags,
                                float *scores, int32_t *anchor_idx, void *y, acache_stream_t stream);

/* Predict-then-commit on the current block (Section 3.1, Eq. 2-3, with the confidence-threshold
 * commit rule the paper's set-up uses, threshold 0.9 in Section 5):
 *   z = W_lm (RMSNorm(h_i) g);  token_i = argmax_v z_v;  conf_i = softmax(z)[token_i]
 *   commit_i = conf_i > threshold; a request none of whose rows qualifies commits its single most
 *   confident row (lowest index on ties).
 * h: DEVICE bf16 [B, h_rows, D], the last layer's compact output; block_rows: DEVICE int32
 * [B, n_blk], the compact row (0 <= . < h_rows) of each masked position of the current block.
 * final_norm_g: DEVICE bf16 [D]; w_lm: DEVICE bf16 [V, D], V a multiple of 128.
 * token, commit: DEVICE int32 [B, n_blk]; confidence: DEVICE fp32 [B, n_blk].
 * Needs batch * n_blk <= max_batch * max_block, V <= max_vocab of the descriptor. */
acache_status acache_predict_commit(acache_ctx *ctx, const void *h, int32_t h_rows, const int32_t *block_rows,
                                    int32_t batch, int32_t n_blk, const void *final_norm_g, const void *w_lm,
                                    int32_t vocab, float threshold, int32_t *token, float *confidence,
                                    int32_t *commit, acache_stream_t stream);

/* One denoising step's model pass for a batch of requests (the "recompute forward" of Section 4.3
 * followed by Eq. 2-3): the rows R = A u E of every request go through n_layers layers, each layer
 * refreshing its cache rows exactly as acache_layer_step(flags = 0) does with the fixed anchor set;
 * the last layer's rows named by block_rows then go through acache_predict_commit.
 *   layers, kvs: HOST arrays of n_layers weight structs / cache descriptors (DEVICE pointers inside).
 *   x0: DEVICE bf16 layer-0 input, [B, ctx_len, D], or the embedding table when req->token_ids is set.
 *   y_a, y_b: DEVICE bf16 [B, K+e, D] each; layer outputs alternate between them, the last layer's
 *             output is in *y_last (HOST pointer to a DEVICE pointer, may be NULL).
 *   block_rows: DEVICE int32 [B, n_blk] compact rows (in [0, K+e)) of the current block's masked positions. */
acache_status acache_denoise_step(acache_ctx *ctx, int32_t n_layers, const acache_layer_weights *layers,
                                  acache_kv *kvs, const acache_request *req, const void *x0,
                                  const int32_t *anchor_idx, int32_t k, void *y_a, void *y_b, void **y_last,
                                  const int32_t *block_rows, int32_t n_blk, const void *final_norm_g,
                                  const void *w_lm, int32_t vocab, float threshold, int32_t *token,
                                  float *confidence, int32_t *commit, acache_stream_t stream);

/* acache_denoise_step over shared affix storage (Section 4.1): the same N-layer refresh of R = A u E and the
 * same predict-then-commit, but no cache is written.  kvs[n] may have batch_stride 0 (one cache per layer
 * for the whole batch); layer n's fresh K/V go to the requests' private slots k_new[n] / v_new[n] (HOST
 * arrays of n_layers DEVICE pointers, each bf16 [B, K+e, Hkv, d]), and layer n's attention reads the
 * positions of R from them and every other position from kvs[n], exactly as acache_recompute_anchors.
 * A later step over the same R can leave the shared caches as they are and keep these slots.
 * Other arguments as acache_denoise_step. */
acache_status acache_denoise_step_shared(acache_ctx *ctx, int32_t n_layers, const acache_layer_weights *layers,
                                         const acache_kv *kvs, const acache_request *req, const void *x0,
                                         const int32_t *anchor_idx, int32_t k, void *const *k_new,
                                         void *const *v_new, void *y_a, void *y_b, void **y_last,
                                         const int32_t *block_rows, int32_t n_blk, const void *final_norm_g,
                                         const void *w_lm, int32_t vocab, float threshold, int32_t *token,
                                         float *confidence, int32_t *commit, acache_stream_t stream);

/* acache_layer_step on storage that is not written (Section 4.1): the cache may be one copy for the
 * whole batch (kv->batch_stride = 0) or one per request; scores and selection read it, and the refreshed
 * K/V of the rows of R go to k_new / v_new (DEVICE bf16 [B, K + e, Hkv, d], the request's private slots)
 * instead of into the cache; their attention reads every other position from the cache.  Equivalent to the
 * masked rows' query projection + acache_score_anchors + acache_select_topk + acache_recompute_anchors.
 * Flags, x, scores, anchor_idx and y as acache_layer_step; k_new / v_new may be NULL only with
 * ACACHE_F_NO_RECOMPUTE. */
acache_status acache_layer_step_shared(acache_ctx *ctx, const acache_layer_weights *w, const acache_request *req,
                                       const acache_kv *kv, const void *x, int x_is_compact, double ratio,
                                       uint32_t flags, float *scores, int32_t *anchor_idx, void *k_new,
                                       void *v_new, void *y, acache_stream_t stream);

/* A decode pass over shared affix storage (Section 4.1 storage under the Section 4.3 schedule): after a
 * refresh pass (acache_recompute_anchors / acache_denoise_step_shared with kv->batch_stride = 0) has
 * filled the private slot arrays k_slots / v_slots [B, k + e_slots, Hkv, d] with the anchors and the
 * request-specific rows of req_slots, this call recomputes only the rows req_rows->extra_rows (n_extra
 * per request: the block being decoded) through one layer.  Their fresh K/V overwrite slot rows
 * slot_rows[b, i] (the index of row i's position inside the slot array: k + its index in
 * req_slots->extra_rows); their attention reads every other position from the shared cache, except
 * those a slot row serves, which come from the slots (the read-slot map of Section 4.1).
 *   req_rows, req_slots: same batch, ctx_len, affix span and rope tables; req_slots, anchor_idx and k as
 *   given to the refresh pass.  x, x_is_compact: as acache_recompute_anchors, for the rows of req_rows.
 *   slot_rows: DEVICE int32 [B, n_extra]; a value outside [0, k + e_slots) raises
 *   ACACHE_FLAG_BAD_INDEX and that row's K/V is not stored.  A position that appears twice in the slot
 *   array is served by its last row; slot_rows must name that one.
 *   k_slots, v_slots: DEVICE bf16, updated in place.  y: DEVICE bf16 [B, n_extra, D].
 * The shared cache is not written. */
acache_status acache_recompute_rows_shared(acache_ctx *ctx, const acache_layer_weights *w,
                                           const acache_request *req_rows, const acache_request *req_slots,
                                           const acache_kv *kv, const void *x, int x_is_compact,
                                           const int32_t *anchor_idx, int32_t k, const int32_t *slot_rows,
                                           void *k_slots, void *v_slots, void *y, acache_stream_t stream);

/* n_layers of acache_recompute_rows_shared chained (layer n reads kvs[n], k_slots[n], v_slots[n]; HOST
 * arrays of DEVICE pointers), then Eq. 2-3 on the rows block_rows of the last layer's output, as
 * acache_denoise_step_shared does for the refresh pass.  y_a, y_b: DEVICE bf16 [B, n_extra, D]. */
acache_status acache_decode_step_shared(acache_ctx *ctx, int32_t n_layers, const acache_layer_weights *layers,
                                        const acache_kv *kvs, const acache_request *req_rows,
                                        const acache_request *req_slots, const void *x0,
                                        const int32_t *anchor_idx, int32_t k, const int32_t *slot_rows,
                                        void *const *k_slots, void *const *v_slots, void *y_a, void *y_b,
                                        void **y_last, const int32_t *block_rows, int32_t n_blk,
                                        const void *final_norm_g, const void *w_lm, int32_t vocab, float threshold,
                                        int32_t *token, float *confidence, int32_t *commit, acache_stream_t stream);

/* acache_generate_block over shared affix storage: step 0 is acache_denoise_step_shared over
 * R = A u E (req_refresh), which fills the private slots; every later step is
 * acache_decode_step_shared over the block's rows (req_decode) with slot_rows = block_rows_refresh.
 * The shared caches kvs[n] (batch_stride 0) are never written; everything a request changes lives in
 * its slots.  Other arguments, the commit rule and the one synchronisation per step as
 * acache_generate_block. */
acache_status acache_generate_block_shared(acache_ctx *ctx, int32_t n_layers, const acache_layer_weights *layers,
                                           const acache_kv *kvs, const acache_request *req_refresh,
                                           const acache_request *req_decode, const void *embed,
                                           const int32_t *anchor_idx, int32_t k, void *const *k_slots,
                                           void *const *v_slots, void *y_a, void *y_b,
                                           const int32_t *block_rows_refresh, const int32_t *block_rows_decode,
                                           int32_t n_blk, const void *final_norm_g, const void *w_lm, int32_t vocab,
                                           float threshold, int32_t mask_id, int32_t max_steps, int32_t *token,
                                           float *confidence, int32_t *commit, int32_t *remaining,
                                           int32_t *steps_done, acache_stream_t stream);

/* The one-shot probe and the selection it feeds (Section 3.2): every request's request-specific rows
 * (req->extra_rows = all non-affix positions, which must include the masked ones) go through the
 * n_layers layers with the affix K/V as cached; at every layer the masked rows' queries are scored
 * against the cached affix keys (Eq. 4) and the scores accumulate over the layers (Eq. 5); then
 * Eq. 6 picks K = acache_k_from_ratio(affix_len, ratio) anchors once for all layers.  Equivalent to
 * n_layers calls of acache_layer_step(ratio 0, ACACHE_F_SCORE [| ACACHE_F_ACCUMULATE]) followed by
 * acache_select_topk; like them it writes the fresh K/V of the request-specific rows into kvs.
 *   flags: 0 or ACACHE_F_SCORE_NORM_FULL.  layers, kvs: HOST arrays (DEVICE pointers inside).
 *   x0: DEVICE bf16 [B, ctx_len, D], or the embedding table when req->token_ids is set.
 *   y_a, y_b: DEVICE bf16 [B, e, D] each (layer outputs alternate between them).
 *   scores: DEVICE fp32 [B, L] (overwritten); anchor_idx: DEVICE int32 [B, K] ascending. */
acache_status acache_probe_select(acache_ctx *ctx, int32_t n_layers, const acache_layer_weights *layers,
                                  acache_kv *kvs, const acache_request *req, const void *x0, double ratio,
                                  uint32_t flags, void *y_a, void *y_b, float *scores, int32_t *anchor_idx,
                                  acache_stream_t stream);

/* Eq. 3 applied to the sequence: among the block's positions block_pos[b, i] whose token id is still
 * mask_id, those with confidence[b, i] > threshold receive token[b, i]; if a request has masked
 * positions but none qualifies, its single most confident masked position does (lowest i on ties).
 * Positions already decoded are left alone whatever their confidence.
 *   token_ids: DEVICE int32 [B, ctx_len], updated in place; block_pos: DEVICE int32 [B, n_blk] absolute
 *   positions; token, confidence: DEVICE [B, n_blk] as written by acache_predict_commit for those rows;
 *   remaining: DEVICE int32 [B], masked positions left in the block after the update.
 * A position outside [0, ctx_len) raises ACACHE_FLAG_BAD_INDEX and is skipped. */
acache_status acache_commit_update(acache_ctx *ctx, int32_t *token_ids, int32_t ctx_len, const int32_t *block_pos,
                                   int32_t batch, int32_t n_blk, const int32_t *token, const float *confidence,
                                   int32_t mask_id, float threshold, int32_t *remaining, acache_stream_t stream);

/* Decoding of one block with the refresh-then-decode schedule of Section 4.3 / Section 5: step 0 is
 * acache_denoise_step over R = A u E (req_refresh: anchors + all request-specific rows), which brings
 * the caches up to date; every later step recomputes only the block's rows (req_decode: k = 0,
 * extra_rows = the block's positions) over the same caches.  After each step acache_commit_update
 * writes the committed tokens into token_ids; the loop ends when no request has a masked position
 * left in the block or after max_steps steps.
 *   Both requests must name the same token_ids (DEVICE int32 [B, ctx_len], updated in place); embed is
 *   the embedding table [n_embed, D].  block_rows_refresh / block_rows_decode: DEVICE int32 [B, n_blk],
 *   the compact row of each block position inside the rows of the refresh / decode pass (the latter
 *   normally 0 .. n_blk-1).  y_a, y_b: DEVICE bf16 [B, K+e, D] sized for the refresh pass.
 *   token, confidence, commit: DEVICE [B, n_blk] (the last step's predictions); remaining: DEVICE [B].
 *   steps_done: HOST, number of model passes run.
 * THIS CALL SYNCHRONISES the stream once per step (it reads `remaining` back, 4 bytes per request). */
acache_status acache_generate_block(acache_ctx *ctx, int32_t n_layers, const acache_layer_weights *layers,
                                    acache_kv *kvs, const acache_request *req_refresh,
                                    const acache_request *req_decode, const void *embed,
                                    const int32_t *anchor_idx, int32_t k, void *y_a, void *y_b,
                                    const int32_t *block_rows_refresh, const int32_t *block_rows_decode,
                                    int32_t n_blk, const void *final_norm_g, const void *w_lm, int32_t vocab,
                                    float threshold, int32_t mask_id, int32_t max_steps, int32_t *token,
                                    float *confidence, int32_t *commit, int32_t *remaining, int32_t *steps_done,
                                    acache_stream_t stream);

/* acache_layer_step for a caller whose per-step data lives in HOST memory: copies
 * x [B, ctx_len, D] (HOST bf16, ideally pinned) to a staging area in the workspace,
 * runs the layer-step with ACACHE_F_SCORE | ACACHE_F_SELECT | flags, and copies y
 * [B, K+e, D], anchor_idx [B, K] and scores [B, L] back to the given HOST buffers.
 * Weights, cache and the request's index arrays stay DEVICE-resident.  All copies are
 * asynchronous on `stream`; the caller synchronises the stream before reading.
 *   When x_host is page-locked (acache_host_x_in_place returns 1) and the step needs at most a quarter of
 *   its rows, it is not staged: the kernels read
 *   the rows the step needs (the masked rows and the K+e recomputed rows: n_masked + K + e rows of D bf16 per
 *   request, each once) in place over the bus, so x_host must stay valid and unchanged until the
 *   stream has passed this call.  Page-locked scores_host / anchor_idx_host are written by a copy kernel. */
acache_status acache_layer_step_host(acache_ctx *ctx, const acache_layer_weights *w,
                                     const acache_request *req, acache_kv *kv,
                                     const void *x_host, double ratio, uint32_t flags,
                                     float *scores_host, int32_t *anchor_idx_host, void *y_host,
                                     acache_stream_t stream);

/* 1 when acache_layer_step_host reads an x at this HOST address in place (page-locked memory the device
 * can address), 0 when it stages a copy.  No GPU work; ACACHE_HOST_X_IN_PLACE=0 in the environment
 * forces 0. */
int32_t acache_host_x_in_place(const void *x_host);

#ifdef __cplusplus
}
#endif
#endif /* ACACHE_H_ */
