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

void launch_build_slot_map(int32_t* slot, int ctx_len, const int32_t* row_pos, int rows_per_req, int batch,
                           cudaStream_t stream) {
    if (batch == 0) return;
    launch_pdl(slot_map_kernel, batch, 1024, 0, stream, slot, ctx_len, row_pos, rows_per_req);
}

}  // namespace acache
