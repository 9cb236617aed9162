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

}  // namespace acache
