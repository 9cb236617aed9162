// Row kernels of the selective recomputation (Section 3.3): the KV scatter (working-cache
// construction) and the position -> fresh-row map used when the cache must not be mutated.
// (Gather + RMSNorm of the rows runs inside the projection kernel, gemm_tc.cu.)
#include "common.cuh"
#include "rows.cuh"
#include "kernels.h"
#include "launch.h"

namespace acache {

__global__ void __launch_bounds__(128) scatter_kv_kernel(
    __nv_bfloat16* __restrict__ cache_k, __nv_bfloat16* __restrict__ cache_v, int64_t batch_stride, int ctx_len,
    const int32_t* __restrict__ anchor_idx, int k, const int32_t* __restrict__ extra_rows, int e,
    int affix_start, int affix_len, int kv_dim, const __nv_bfloat16* __restrict__ k_new,
    const __nv_bfloat16* __restrict__ v_new, uint32_t* status) {
    pdl_wait();
    pdl_launch_dependents();
    const int rows_per_req = k + e;
    const int row = blockIdx.x;
    const int b = row / rows_per_req, i = row - b * rows_per_req;
    const int pos = row_position(anchor_idx, k, extra_rows, e, b, i, affix_start, affix_len, ctx_len);
    if (pos < 0) {
        if (threadIdx.x == 0) atomicOr(status, kFlagBadIndex);
        return;
    }
    const int nchunk = kv_dim >> 3;
    const uint4* sk = reinterpret_cast<const uint4*>(k_new + (int64_t)row * kv_dim);
    const uint4* sv = reinterpret_cast<const uint4*>(v_new + (int64_t)row * kv_dim);
    uint4* dk = reinterpret_cast<uint4*>(cache_k + (int64_t)b * batch_stride + (int64_t)pos * kv_dim);
    uint4* dv = reinterpret_cast<uint4*>(cache_v + (int64_t)b * batch_stride + (int64_t)pos * kv_dim);
    for (int c = threadIdx.x; c < nchunk; c += blockDim.x) {
        dk[c] = sk[c];
        dv[c] = sv[c];
    }
}

__global__ void __launch_bounds__(1024) slot_map_kernel(int32_t* __restrict__ slot, int ctx_len,
                                                        const int32_t* __restrict__ row_pos, int rows_per_req) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x;
    int32_t* s = slot + (int64_t)b * ctx_len;
    for (int t = threadIdx.x; t < ctx_len; t += blockDim.x) s[t] = -1;
    __syncthreads();
    // later rows win on duplicates, the same order a sequential scatter would give
    if (threadIdx.x == 0) {
        for (int i = 0; i < rows_per_req; ++i) {
            int p = row_pos[(int64_t)b * rows_per_req + i];
            if (p >= 0) s[p] = i;
        }
    }
}

// Bit masks over keys for the attention that reads the cache and the fresh rows as two sources
// (Section 4.1: shared storage + private slots): pos_excl[b] bit t = position t is served by a fresh
// row (skip it in the cache); row_keep[b] bit i = fresh row i is the one that serves its position
// (the last one wins if two rows name the same position, as in the position -> row map).
__global__ void __launch_bounds__(1024) key_mask_kernel(const int32_t* __restrict__ slot, int ctx_len,
                                                        const int32_t* __restrict__ row_pos, int rows_per_req,
                                                        uint32_t* __restrict__ pos_excl, int excl_words,
                                                        uint32_t* __restrict__ row_keep, int keep_words) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    const int32_t* s = slot + (int64_t)b * ctx_len;
    for (int w = warp; w < excl_words; w += nw) {
        const int t = w * 32 + lane;
        const uint32_t bits = __ballot_sync(0xffffffffu, t < ctx_len && s[t] >= 0);
        if (lane == 0) pos_excl[(int64_t)b * excl_words + w] = bits;
    }
    for (int w = warp; w < keep_words; w += nw) {
        const int i = w * 32 + lane;
        bool ok = false;
        if (i < rows_per_req) {
            const int p = row_pos[(int64_t)b * rows_per_req + i];
            ok = p >= 0 && p < ctx_len && s[p] == i;
        }
        const uint32_t bits = __ballot_sync(0xffffffffu, ok);
        if (lane == 0) row_keep[(int64_t)b * keep_words + w] = bits;
    }
}

void launch_key_masks(const int32_t* slot, int ctx_len, const int32_t* row_pos, int rows_per_req, int batch,
                      uint32_t* pos_excl, int excl_words, uint32_t* row_keep, int keep_words, cudaStream_t stream) {
    if (batch == 0) return;
    launch_pdl(key_mask_kernel, batch, 1024, 0, stream, slot, ctx_len, row_pos, rows_per_req, pos_excl, excl_words, row_keep,
               keep_words);
}

// idx[b, i] = k + j where extra_rows[b, j] == masked_pos[b, i]: the compact row that holds a
// masked position when the layer input is given in compact row order; -1 (and kFlagBadIndex)
// if the position is not among the extra rows.
__global__ void __launch_bounds__(256) match_rows_kernel(const int32_t* __restrict__ masked_pos, int m,
                                                         const int32_t* __restrict__ extra_rows, int e, int k,
                                                         int32_t* __restrict__ idx, uint32_t* status) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= m) return;
    const int want = masked_pos[(int64_t)b * m + i];
    int found = -1;
    for (int j = 0; j < e; ++j)
        if (extra_rows[(int64_t)b * e + j] == want) { found = k + j; break; }
    idx[(int64_t)b * m + i] = found;
    if (found < 0) atomicOr(status, kFlagBadIndex);
}

// Eq. 3 on the sequence state: among the block's positions that still hold the mask id, those whose
// confidence exceeds the threshold receive their predicted token; if none does, the single most
// confident one (lowest index on ties).  One warp per request; remaining[b] = masked positions left.
__global__ void __launch_bounds__(32) commit_update_kernel(int32_t* __restrict__ token_ids, int ctx_len,
                                                           const int32_t* __restrict__ block_pos, int n_blk,
                                                           const int32_t* __restrict__ token,
                                                           const float* __restrict__ confidence, int mask_id,
                                                           float threshold, int32_t* __restrict__ remaining,
                                                           uint32_t* __restrict__ status) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, lane = threadIdx.x;
    int32_t* ids = token_ids + (int64_t)b * ctx_len;
    int n_masked = 0, n_commit = 0, best_i = -1;
    float best_c = -INFINITY;
    for (int i0 = 0; i0 < n_blk; i0 += 32) {
        const int i = i0 + lane;
        bool masked = false, hit = false;
        float c = -INFINITY;
        int pos = 0;
        if (i < n_blk) {
            pos = block_pos[(int64_t)b * n_blk + i];
            if (pos < 0 || pos >= ctx_len) {
                atomicOr(status, kFlagBadIndex);
            } else {
                masked = ids[pos] == mask_id;
                c = confidence[(int64_t)b * n_blk + i];
                hit = masked && c > threshold;
                if (hit) ids[pos] = token[(int64_t)b * n_blk + i];
            }
        }
        n_masked += __popc(__ballot_sync(0xffffffffu, masked));
        n_commit += __popc(__ballot_sync(0xffffffffu, hit));
        // most confident masked row of this chunk, lowest index on ties
        float cc = masked ? c : -INFINITY;
        int ci = masked ? i : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float oc = __shfl_xor_sync(0xffffffffu, cc, o);
            const int oi = __shfl_xor_sync(0xffffffffu, ci, o);
            if (oc > cc || (oc == cc && oi < ci)) { cc = oc; ci = oi; }
        }
        if (ci != 0x7fffffff && (cc > best_c || best_i < 0)) { best_c = cc; best_i = ci; }
    }
    if (n_commit == 0 && n_masked > 0 && best_i >= 0) {
        if (lane == 0) ids[block_pos[(int64_t)b * n_blk + best_i]] = token[(int64_t)b * n_blk + best_i];
        n_commit = 1;
    }
    if (lane == 0) remaining[b] = n_masked - n_commit;
}

void launch_commit_update(int32_t* token_ids, int ctx_len, const int32_t* block_pos, int batch, int n_blk,
                          const int32_t* token, const float* confidence, int mask_id, float threshold,
                          int32_t* remaining, uint32_t* status, cudaStream_t stream) {
    if (batch == 0) return;
    launch_pdl(commit_update_kernel, dim3(batch), dim3(32), 0, stream, token_ids, ctx_len, block_pos, n_blk, token, confidence,
               mask_id, threshold, remaining, status);
}

void launch_match_rows(const int32_t* masked_pos, int m, const int32_t* extra_rows, int e, int k, int batch,
                       int32_t* idx, uint32_t* status, cudaStream_t stream) {
    if (batch == 0 || m == 0) return;
    launch_pdl(match_rows_kernel, dim3((m + 255) / 256, batch), dim3(256), 0, stream, masked_pos, m, extra_rows, e, k, idx,
               status);
}

void launch_scatter_kv(void* cache_k, void* cache_v, int64_t batch_stride, int ctx_len, const int32_t* anchor_idx,
                       int k, const int32_t* extra_rows, int e, int batch, int affix_start, int affix_len,
                       int kv_dim, const void* k_new, const void* v_new, uint32_t* status, cudaStream_t stream) {
    const int n = batch * (k + e);
    if (n == 0) return;
    launch_pdl(scatter_kv_kernel, n, 128, 0, stream, static_cast<__nv_bfloat16*>(cache_k),
                                             static_cast<__nv_bfloat16*>(cache_v), batch_stride, ctx_len,
                                             anchor_idx, k, extra_rows, e, affix_start, affix_len, kv_dim,
                                             static_cast<const __nv_bfloat16*>(k_new),
                                             static_cast<const __nv_bfloat16*>(v_new), status);
}

// row_pos[b, i] = position of private row i of request b (anchors first, then the extra rows); -1 and
// kFlagBadIndex for an index out of range.
__global__ void __launch_bounds__(256) row_pos_kernel(const int32_t* __restrict__ anchor_idx, int k,
                                                      const int32_t* __restrict__ extra_rows, int e, int affix_start,
                                                      int affix_len, int ctx_len, int32_t* __restrict__ row_pos,
                                                      uint32_t* status) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.y, i = blockIdx.x * 256 + threadIdx.x;
    if (i >= k + e) return;
    const int pos = row_position(anchor_idx, k, extra_rows, e, b, i, affix_start, affix_len, ctx_len);
    if (pos < 0) atomicOr(status, kFlagBadIndex);
    row_pos[(int64_t)b * (k + e) + i] = pos;
}

void launch_row_positions(const int32_t* anchor_idx, int k, const int32_t* extra_rows, int e, int affix_start, int affix_len,
                          int ctx_len, int batch, int32_t* row_pos, uint32_t* status, cudaStream_t stream) {
    if (batch == 0 || k + e == 0) return;
    launch_pdl(row_pos_kernel, dim3((k + e + 255) / 256, batch), dim3(256), 0, stream, anchor_idx, k, extra_rows, e, affix_start,
               affix_len, ctx_len, row_pos, status);
}

void launch_build_slot_map(int32_t* slot, int ctx_len, const int32_t* row_pos, int rows_per_req, int batch,
                           cudaStream_t stream) {
    if (batch == 0) return;
    launch_pdl(slot_map_kernel, batch, 1024, 0, stream, slot, ctx_len, row_pos, rows_per_req);
}

// ---- KV-deviation selector (the CacheBlend-style variant of the paper's appendix) ------------------
// scores[b, j] (+)= sum over the KV heads and the head dimension of (K_full - K_ref)^2 + (V_full - V_ref)^2
// at affix token j.  One CTA per (token, request): the four rows are streamed once with 16-byte loads,
// squared differences accumulate in fp32, and the block sum runs in a fixed order (bitwise reproducible).
__global__ void __launch_bounds__(128) kv_deviation_kernel(const __nv_bfloat16* __restrict__ k_ref,
                                                           const __nv_bfloat16* __restrict__ v_ref, int64_t ref_stride,
                                                           const __nv_bfloat16* __restrict__ k_full,
                                                           const __nv_bfloat16* __restrict__ v_full, int64_t full_stride,
                                                           int affix_start, int affix_len, int kv_dim,
                                                           float* __restrict__ scores, int accumulate) {
    __shared__ float red[4];
    pdl_wait();
    pdl_launch_dependents();
    const int j = blockIdx.x, b = blockIdx.y;
    const int64_t row = (int64_t)(affix_start + j) * kv_dim;
    const uint4* src[4] = {reinterpret_cast<const uint4*>(k_ref + (int64_t)b * ref_stride + row),
                           reinterpret_cast<const uint4*>(k_full + (int64_t)b * full_stride + row),
                           reinterpret_cast<const uint4*>(v_ref + (int64_t)b * ref_stride + row),
                           reinterpret_cast<const uint4*>(v_full + (int64_t)b * full_stride + row)};
    const int nchunk = kv_dim >> 3;
    float acc = 0.f;
    for (int c0 = threadIdx.x; c0 < nchunk; c0 += 4 * 128) {
        uint4 u[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = c0 + i * 128;
#pragma unroll
            for (int t = 0; t < 4; ++t) u[i][t] = c < nchunk ? __ldcs(src[t] + c) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int t = 0; t < 4; t += 2) {
                const uint32_t a[4] = {u[i][t].x, u[i][t].y, u[i][t].z, u[i][t].w};
                const uint32_t f[4] = {u[i][t + 1].x, u[i][t + 1].y, u[i][t + 1].z, u[i][t + 1].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float d0 = bf16_lo(f[e]) - bf16_lo(a[e]), d1 = bf16_hi(f[e]) - bf16_hi(a[e]);
                    acc = fmaf(d0, d0, acc);
                    acc = fmaf(d1, d1, acc);
                }
            }
    }
    const float tot = block_sum(acc, red);
    if (threadIdx.x == 0) {
        float* out = scores + (int64_t)b * affix_len + j;
        *out = accumulate ? *out + tot : tot;
    }
}

void launch_kv_deviation(const void* k_ref, const void* v_ref, int64_t ref_stride, const void* k_full, const void* v_full,
                         int64_t full_stride, int affix_start, int affix_len, int kv_dim, int batch, float* scores,
                         int accumulate, cudaStream_t stream) {
    if (batch == 0 || affix_len == 0) return;
    launch_pdl(kv_deviation_kernel, dim3(affix_len, batch), dim3(128), 0, stream, static_cast<const __nv_bfloat16*>(k_ref),
               static_cast<const __nv_bfloat16*>(v_ref), ref_stride, static_cast<const __nv_bfloat16*>(k_full),
               static_cast<const __nv_bfloat16*>(v_full), full_stride, affix_start, affix_len, kv_dim, scores, accumulate);
}

// ---- DropNA layout (Section 5.3): the non-anchor affix entries do not exist as keys ------------------
// key_drop[b] bit t = position t lies in the affix and is not one of request b's anchors.  With or_into the same
// bits are also OR-ed into the cache-exclusion mask of the two-source attention (there the anchors come from
// the fresh rows, so the whole affix span of the cache is skipped).
__global__ void __launch_bounds__(256) drop_mask_kernel(const int32_t* __restrict__ anchor_idx, int k, int affix_start,
                                                        int affix_len, int ctx_len, uint32_t* __restrict__ key_drop,
                                                        uint32_t* __restrict__ or_into, int words) {
    extern __shared__ uint32_t bits[];
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x;
    for (int w = threadIdx.x; w < words; w += blockDim.x) {
        const int lo = max(affix_start - w * 32, 0), hi = min(affix_start + affix_len - w * 32, 32);
        uint32_t m = 0u;
        if (hi > lo) m = (hi - lo >= 32 ? 0xffffffffu : ((1u << (hi - lo)) - 1u) << lo);
        bits[w] = m;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < k; i += blockDim.x) {
        const int a = anchor_idx[(int64_t)b * k + i];
        if (a >= 0 && a < affix_len) {
            const int t = affix_start + a;
            atomicAnd(&bits[t >> 5], ~(1u << (t & 31)));
        }
    }
    __syncthreads();
    for (int w = threadIdx.x; w < words; w += blockDim.x) {
        key_drop[(int64_t)b * words + w] = bits[w];
        if (or_into) or_into[(int64_t)b * words + w] |= bits[w];
    }
}

void launch_drop_mask(const int32_t* anchor_idx, int k, int affix_start, int affix_len, int ctx_len, int batch,
                      uint32_t* key_drop, uint32_t* or_into, int words, cudaStream_t stream) {
    if (batch == 0) return;
    launch_pdl(drop_mask_kernel, dim3(batch), dim3(256), (size_t)words * sizeof(uint32_t), stream, anchor_idx, k, affix_start,
               affix_len, ctx_len, key_drop, or_into, words);
}

// ---- Eq. 4-5 from the probe's own attention logits: which compact rows are masked positions, and the final sum --------
__global__ void __launch_bounds__(256) row_mask_kernel(const int32_t* __restrict__ masked_pos, int m,
                                                       const int32_t* __restrict__ extra_rows, int e, int k,
                                                       uint32_t* __restrict__ rowmask, int words, uint32_t* status) {
    extern __shared__ uint32_t bits[];          // [words] the mask, then [e] the request's extra rows
    int32_t* rows_s = reinterpret_cast<int32_t*>(bits + words);
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x;
    for (int w = threadIdx.x; w < words; w += blockDim.x) bits[w] = 0u;
    for (int j = threadIdx.x; j < e; j += blockDim.x) rows_s[j] = extra_rows[(int64_t)b * e + j];
    __syncthreads();
    for (int i = threadIdx.x; i < m; i += blockDim.x) {
        const int want = masked_pos[(int64_t)b * m + i];
        int found = -1;
        for (int j = 0; j < e; ++j)
            if (rows_s[j] == want) { found = k + j; break; }
        if (found < 0 || (found >> 5) >= words) atomicOr(status, kFlagBadIndex);
        else atomicOr(&bits[found >> 5], 1u << (found & 31));
    }
    __syncthreads();
    for (int w = threadIdx.x; w < words; w += blockDim.x) rowmask[(int64_t)b * words + w] = bits[w];
}

void launch_row_mask(const int32_t* masked_pos, int m, const int32_t* extra_rows, int e, int k, int batch, uint32_t* rowmask,
                     int words, uint32_t* status, cudaStream_t stream) {
    if (batch == 0) return;
    const size_t smem = (size_t)(words + e) * sizeof(uint32_t);
    if (smem > 48 * 1024) cudaFuncSetAttribute(row_mask_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    launch_pdl(row_mask_kernel, dim3(batch), dim3(256), smem, stream, masked_pos, m, extra_rows, e, k, rowmask, words, status);
}

// Two small results of a step (scores, anchor indices: 4-byte words) copied to page-locked host memory by plain
// stores over the bus, one launch instead of two copy-engine transfers.
__global__ void __launch_bounds__(256) copy_out_words_kernel(const uint32_t* __restrict__ a, uint32_t* __restrict__ a_out, int n_a,
                                                             const uint32_t* __restrict__ b, uint32_t* __restrict__ b_out, int n_b) {
    pdl_wait();
    pdl_launch_dependents();
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_a + n_b; i += gridDim.x * blockDim.x) {
        if (i < n_a) a_out[i] = a[i];
        else b_out[i - n_a] = b[i - n_a];
    }
}

void launch_copy_out_words(const void* a, void* a_out, int n_a, const void* b, void* b_out, int n_b, cudaStream_t stream) {
    if (n_a + n_b <= 0) return;
    const int blocks = (n_a + n_b + 255) / 256;
    launch_pdl(copy_out_words_kernel, dim3(blocks < 148 ? blocks : 148), dim3(256), 0, stream, static_cast<const uint32_t*>(a),
               static_cast<uint32_t*>(a_out), n_a, static_cast<const uint32_t*>(b), static_cast<uint32_t*>(b_out), n_b);
}

__global__ void __launch_bounds__(256) score_reduce_tiles_kernel(const float* __restrict__ partial,
                                                                 const uint32_t* __restrict__ rowmask, int rm_words,
                                                                 float* __restrict__ scores, int n_heads, int q_tiles, int L,
                                                                 int accumulate) {
    __shared__ int live[256];                    // the query tiles that hold a flagged row (they wrote their partial sums)
    __shared__ int n_live;
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.y;
    if (threadIdx.x == 0) {
        int n = 0;
        for (int qt = 0; qt < q_tiles && qt < 256; ++qt) {
            uint32_t any = 0u;
            for (int w = qt * 4; w < min(qt * 4 + 4, rm_words); ++w) any |= rowmask[(int64_t)b * rm_words + w];
            if (any) live[n++] = qt;
        }
        n_live = n;
    }
    __syncthreads();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= L) return;
    // (head, live tile) pairs in a fixed order, eight loads in flight at a time
    const int total = n_heads * n_live;
    float s = 0.f;
    for (int i0 = 0; i0 < total; i0 += 8) {
        float t[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + u;
            t[u] = 0.f;
            if (i < total) {
                const int h = i / n_live, qt = live[i - h * n_live];
                t[u] = __ldcg(partial + (((int64_t)b * n_heads + h) * q_tiles + qt) * L + j);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) s += t[u];
    }
    float* out = scores + (int64_t)b * L + j;
    *out = accumulate ? *out + s : s;
}

void launch_score_reduce_tiles(const float* partial, const uint32_t* rowmask, int rm_words, float* scores, int batch, int n_heads,
                               int q_tiles, int affix_len, int accumulate, cudaStream_t stream) {
    if (batch == 0 || affix_len == 0) return;
    launch_pdl(score_reduce_tiles_kernel, dim3((affix_len + 255) / 256, batch), dim3(256), 0, stream, partial, rowmask, rm_words,
               scores, n_heads, q_tiles, affix_len, accumulate);
}

}  // namespace acache
