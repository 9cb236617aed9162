// Host-side launchers of the CUDA kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace acache {

// ---- rows.cu ----------------------------------------------------------------------------
// cache[b, pos_r] = new[b, r] for K and V; rows with an invalid position are skipped.
void launch_scatter_kv(void* cache_k, void* cache_v, int64_t batch_stride, int ctx_len,
                       const int32_t* anchor_idx, int k, const int32_t* extra_rows, int e, int batch,
                       int affix_start, int affix_len, int kv_dim, const void* k_new, const void* v_new,
                       uint32_t* status, cudaStream_t stream);

// idx[b, i] = compact row (k + j) whose position extra_rows[b, j] equals masked_pos[b, i], or -1.
void launch_match_rows(const int32_t* masked_pos, int m, const int32_t* extra_rows, int e, int k, int batch,
                       int32_t* idx, uint32_t* status, cudaStream_t stream);

// Eq. 3 on the sequence state: the block's still-masked positions whose confidence exceeds the threshold
// (else the single most confident one) receive their predicted token; remaining[b] = masked positions left.
void launch_commit_update(int32_t* token_ids, int ctx_len, const int32_t* block_pos, int batch, int n_blk,
                          const int32_t* token, const float* confidence, int mask_id, float threshold,
                          int32_t* remaining, uint32_t* status, cudaStream_t stream);

// slot[b, t] = compact row index whose fresh K/V replaces position t, or -1.
// Positions of the rows of a private slot array (k anchors, then e extra rows per request).
void launch_row_positions(const int32_t* anchor_idx, int k, const int32_t* extra_rows, int e, int affix_start, int affix_len,
                          int ctx_len, int batch, int32_t* row_pos, uint32_t* status, cudaStream_t stream);
void launch_build_slot_map(int32_t* slot, int ctx_len, const int32_t* row_pos, int rows_per_req, int batch,
                           cudaStream_t stream);

// pos_excl[b, t / 32] bit t % 32 = position t is served by a fresh row; row_keep[b, i / 32] bit i % 32 = fresh
// row i serves its position (built from the position -> row map, so duplicates resolve the same way).
void launch_key_masks(const int32_t* slot, int ctx_len, const int32_t* row_pos, int rows_per_req, int batch,
                      uint32_t* pos_excl, int excl_words, uint32_t* row_keep, int keep_words, cudaStream_t stream);

// scores[b, j] (+)= ||K_full[b, l + j] - K_ref[b, l + j]||^2 + ||V_full[b, l + j] - V_ref[b, l + j]||^2 (batch strides in
// elements, 0 = one cache shared by the batch).
void launch_kv_deviation(const void* k_ref, const void* v_ref, int64_t ref_stride, const void* k_full, const void* v_full,
                         int64_t full_stride, int affix_start, int affix_len, int kv_dim, int batch, float* scores,
                         int accumulate, cudaStream_t stream);

// key_drop[b, t / 32] bit t % 32 = position t is an affix position that is not an anchor of request b (the DropNA
// layout: such keys do not exist); or_into (optional, same shape) receives the same bits by OR.
void launch_drop_mask(const int32_t* anchor_idx, int k, int affix_start, int affix_len, int ctx_len, int batch,
                      uint32_t* key_drop, uint32_t* or_into, int words, cudaStream_t stream);

// rowmask[b, i / 32] bit i % 32 = compact row i (k anchors, then the e extra rows) of request b is one of its masked
// positions; a masked position that is not among the extra rows raises kFlagBadIndex.
void launch_row_mask(const int32_t* masked_pos, int m, const int32_t* extra_rows, int e, int k, int batch, uint32_t* rowmask,
                     int words, uint32_t* status, cudaStream_t stream);

// scores[b, j] (+)= sum over heads and over the query tiles that hold a flagged row of partial[b, h, qt, j], in a fixed order.
void launch_score_reduce_tiles(const float* partial, const uint32_t* rowmask, int rm_words, float* scores, int batch, int n_heads,
                               int q_tiles, int affix_len, int accumulate, cudaStream_t stream);

// a_out[0, n_a) = a, b_out[0, n_b) = b (4-byte words); the outputs may be page-locked host memory seen from the device.
void launch_copy_out_words(const void* a, void* a_out, int n_a, const void* b, void* b_out, int n_b, cudaStream_t stream);

// ---- score.cu ---------------------------------------------------------------------------
struct ScoreArgs {
    const void* q_mask;       // bf16 [B, m, H, d]
    const void* cache_k;      // bf16 [B, cap, Hkv, d]
    int64_t kv_batch_stride;  // elements
    int batch, m, n_heads, n_kv_heads, head_dim;
    int affix_start, affix_len;
    int norm_lo, norm_len;    // key range of the softmax normaliser
    float* row_stats;         // [B, H, n_split, m, 2]
    float* head_partial;      // [B, H, L]
    float* scores;            // [B, L]
    int accumulate;
    int defer_head_sum;       // leave head_partial unsummed: launch_topk(.., head_partial) does it
    uint32_t* status;         // device status word (bounded waits of the tensor-core kernels); may be null
    int early_k;              // the cache was last written at least two kernels back on this stream: its first
                              // key tiles may be requested before the wait for the producer of q_mask
};
// tcgen05 kernels for head dimension 128 and up to 256 masked rows (two passes into row_stats / head_partial);
// 0 = not applicable, -1 = launch failed.  Their statistics use one entry per score_tc_splits() keys.
int launch_score_tc(const ScoreArgs& a, uint32_t* status, cudaStream_t stream);
int score_tc_splits(int norm_len);
int score_num_splits(int norm_len);
int launch_score(const ScoreArgs& a, cudaStream_t stream);  // returns number of kernels launched

// ---- topk.cu ----------------------------------------------------------------------------
// head_partial != null: first scores[b, j] = (accumulate ? scores[b, j] : 0) + sum_h head_partial[b, h, j]
// (ordered sum), then the selection runs on the result.
void launch_topk(float* scores, int batch, int affix_len, int k, int32_t* anchor_idx, const float* head_partial,
                 int n_heads, int accumulate, cudaStream_t stream);

// ---- gemm.cu ----------------------------------------------------------------------------
enum GemmEpilogue : int {
    kEpiQKV = 0,     // bias + RoPE on q/k segments, bf16 stores to q / k_new / v_new (+ optional cache scatter)
    kEpiResidual,    // out = bf16(resid[row] + acc)
    kEpiSwiGLU,      // out = bf16(silu(gate) * up); B tile = 128 gate rows + 128 up rows
    kEpiLogits,      // no tensor out: per (row, tile[, 16-column item]) softmax statistics (max, sum exp, argmax)
};

// Row plan of the recompute set R and RMSNorm of the gathered rows, run in front of a GEMM:
// row i of request b (i < k: anchor, else extra) sits at absolute position pos; writes
// row_pos[b*(k+e)+i] = pos (-1 for an out-of-range index, which also raises kFlagBadIndex),
// row_src = element offset of the row inside x, and the GEMM's A rows
// xn = bf16(x * rsqrt(mean(x^2) + eps) * g).
struct RowPrep {
    int enabled;              // 0: off, 1: gather the rows of R, 2: the rows of x as they are (compact),
                              // 3: compact rows picked by compact_idx (no positions)
    const void* x;            // bf16 [B, ctx_len, hidden] or compact [B, k+e, hidden]
    int x_is_compact;
    int64_t x_batch_stride;
    const int32_t* token_ids;    // optional [B, ctx_len]: x is an embedding table [table_rows, hidden] indexed by token id
    int table_rows;
    const int32_t* compact_idx;  // optional [B, k+e]: row i reads compact row compact_idx[..] of its request
    int compact_rows;            // rows per request of the compact x that compact_idx points into
    const int32_t* anchor_idx;
    int k;
    const int32_t* extra_rows;
    int e;
    int affix_start, affix_len, ctx_len;
    const void* gain;
    float eps;
    void* raw_out;            // optional bf16 [M, K]: the gathered rows as read (x far away, e.g. in host memory: read it once)
    int32_t* row_pos;
    int64_t* row_src;
};
struct GemmArgs {
    const void* a;            // bf16 [M, K] row-major, lda = K
    int M, K;
    // B operand: up to three [N_i, K] row-major weight matrices laid side by side along N
    const void* b[3];
    int n[3];
    int epilogue;
    // --- kEpiQKV ---
    const void* bias[3];      // bf16 [N_i] or null
    const int32_t* row_pos;   // [M] absolute position per row (RoPE angle, scatter target); -1 = invalid
    const float* rope_cos;    // [T, d/2]
    const float* rope_sin;
    int head_dim;
    int rope_segments;        // number of leading segments that get RoPE (q only: 1, q+k: 2)
    void* out[3];             // compact bf16 [M, N_i] per segment (may be null)
    void* cache_k;            // optional fused scatter targets for segments 1 and 2
    void* cache_v;
    int64_t kv_batch_stride;
    int rows_per_req;
    // optional: row i of the k/v segments goes to row kv_out_rows[i] of its request's kv_out_stride rows of
    // out[1] / out[2] (a decode pass refreshing some rows of a larger private slot array) instead of row i
    const int32_t* kv_out_rows;
    int kv_out_stride;
    // the weights are read again by the next projection (the masked rows' queries before Q/K/V): keep them in L2
    int keep_weights;
    // K blocks past the ring asked into L2 before the dependency wait (0: the default; worth it only behind a long
    // kernel that leaves memory idle)
    int prefetch_blocks;
    // failure-detection self-test: the grid barrier of the row-preparation phase is given a target it cannot reach
    int debug_expire;
    // --- kEpiResidual ---
    const void* resid;        // bf16 base pointer
    const int64_t* resid_off; // [M] element offset of the residual row, or null => row * N
    // --- kEpiSwiGLU / kEpiResidual output ---
    void* c;                  // bf16 [M, Nout]
    // --- kEpiLogits ---
    float4* logit_stats;      // [M, n_tiles, 16] of (max, sum exp(z - max), argmax as int bits, -)
    // --- row work fused in front of the contraction ---
    RowPrep prep;             // writes the A rows (a) before the contraction
    // --- scratch ---
    float* partial;           // fp32 partial tiles, gemm_partial_bytes() of them
    uint32_t* status;         // device status word
    unsigned int* grid_bar;   // two zero-initialised words for the kernel's grid barriers
};
// Bytes of fp32 partial-tile scratch a GEMM of M rows, reduction length K and n_total output
// columns (SwiGLU: the MLP width) needs.
size_t gemm_partial_bytes(int M, int K, int n_total, bool swiglu);
int launch_gemm(const GemmArgs& g, cudaStream_t stream);      // kernels launched, or -1 if a launch failed

// Softmax confidence and arg max of every row from the statistics a kEpiLogits GEMM left
// (launch_gemm must have run with the same M, K, n_total), then the commit rule per request:
// commit[b, i] = conf > threshold, and if no row of request b qualifies, its most confident row.
int launch_predict_commit(const GemmArgs& g, int batch, int n_blk, float threshold, int32_t* token, float* confidence,
                          int32_t* commit, cudaStream_t stream);

// ---- attn.cu ----------------------------------------------------------------------------
struct AttnArgs {
    const void* q;            // bf16 [B, n, H, d] compact
    const void* cache_k;      // bf16 [B, cap, Hkv, d]
    const void* cache_v;
    int64_t kv_batch_stride;
    const void* k_new;        // bf16 [B, n_fresh, Hkv, d] or null
    const void* v_new;
    int n_fresh;              // rows per request in k_new / v_new; 0 = n (the rows being recomputed are the fresh rows)
    const int32_t* slot;      // [B, ctx_len] or null: >= 0 => read k_new/v_new row slot
    const uint32_t* pos_excl; // optional key masks of the same map (launch_key_masks): with them the tensor-core
    const uint32_t* row_keep; //   kernel reads the cache and k_new / v_new as two key sources instead of gathering
    int excl_words, keep_words;
    const uint32_t* key_drop; // optional [B, excl_words]: bit t = position t does not exist as a key (DropNA, Section 5.3)
    // optional (head dimension 128): Eq. 4-5 from this attention's own logits.  score_rowmask [B, rm_words]: bit i = compact
    // row i is a masked position; score_partial [B, H, ceil(n / 128), L]: per (head, query tile) column sums over the affix
    // keys, written by the query tiles that hold a flagged row (launch_score_reduce_tiles adds them up)
    const uint32_t* score_rowmask;
    float* score_partial;
    int rm_words, affix_start, affix_len;
    int score_norm_full;      // the weights' denominator: this attention's own (all keys) instead of the affix keys only
    int batch, n, ctx_len, n_heads, n_kv_heads, head_dim;
    void* o;                  // bf16 [B, n, H*d]
    float* part_o;            // scratch for key splits: fp32 [B*n*H, n_split, d]
    float* part_ml;           // scratch for key splits: fp32 [B*n*H, n_split, 2] (max, denominator)
    uint32_t* status;         // device status word
};
// tcgen05 kernel (head_dim 128; the cache read in place, or cache + fresh rows as two key sources when the
// key masks are given); 0 = not applicable.
int launch_attention_tc(const AttnArgs& a, uint32_t* status, cudaStream_t stream);
size_t attention_scratch_bytes(int head_dim);   // bytes for part_o followed by part_ml
int launch_attention(const AttnArgs& a, cudaStream_t stream);

}  // namespace acache
