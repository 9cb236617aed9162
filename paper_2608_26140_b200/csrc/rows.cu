// Row kernels of the selective recomputation (Section 3.3): the row plan of R = A u E,
// RMSNorm of the gathered rows, the KV scatter (working-cache construction) and the
// position -> fresh-row map used when the cache must not be mutated.
#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace acache {

// Position of compact row i of request b; -1 if the index is out of range.
__device__ __forceinline__ int row_position(const int32_t* anchor_idx, int k, const int32_t* extra_rows, int e,
                                            int b, int i, int affix_start, int affix_len, int ctx_len) {
    if (i < k) {
        int a = anchor_idx[(int64_t)b * k + i];
        if (a < 0 || a >= affix_len) return -1;
        return affix_start + a;
    }
    int p = extra_rows[(int64_t)b * e + (i - k)];
    if (p < 0 || p >= ctx_len) return -1;
    return p;
}

__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < nw; ++i) t += red[i];   // fixed order: bitwise reproducible
    __syncthreads();
    return t;
}

__device__ __forceinline__ void rmsnorm_row(const uint4* __restrict__ xr, const uint4* __restrict__ g,
                                            uint4* __restrict__ out, int hidden, float eps, float* red) {
    const int nchunk = hidden >> 3;
    float ss = 0.f;
    for (int c = threadIdx.x; c < nchunk; c += blockDim.x) {
        uint4 u = xr[c];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float a = bf16_lo(w[i]), b = bf16_hi(w[i]);
            ss += a * a + b * b;
        }
    }
    float tot = block_sum(ss, red);
    float rstd = rsqrtf(tot / (float)hidden + eps);
    for (int c = threadIdx.x; c < nchunk; c += blockDim.x) {
        uint4 u = xr[c], gg = g[c];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
        const uint32_t gw[4] = {gg.x, gg.y, gg.z, gg.w};
        uint32_t r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            r[i] = pack_bf16(bf16_lo(w[i]) * rstd * bf16_lo(gw[i]), bf16_hi(w[i]) * rstd * bf16_hi(gw[i]));
        out[c] = make_uint4(r[0], r[1], r[2], r[3]);
    }
}

__global__ void __launch_bounds__(256) gather_rmsnorm_kernel(
    const __nv_bfloat16* __restrict__ x, int x_is_compact, int64_t x_batch_stride, int hidden,
    const int32_t* __restrict__ anchor_idx, int k, const int32_t* __restrict__ extra_rows, int e,
    int affix_start, int affix_len, int ctx_len, const __nv_bfloat16* __restrict__ gain, float eps,
    int32_t* __restrict__ row_pos, int64_t* __restrict__ row_src, __nv_bfloat16* __restrict__ xn,
    uint32_t* status) {
    __shared__ float red[8];
    pdl_wait();
    pdl_launch_dependents();
    const int rows_per_req = k + e;
    const int row = blockIdx.x;
    const int b = row / rows_per_req, i = row - b * rows_per_req;
    int pos = row_position(anchor_idx, k, extra_rows, e, b, i, affix_start, affix_len, ctx_len);
    int64_t src;
    if (x_is_compact) src = (int64_t)row * hidden;
    else src = (int64_t)b * x_batch_stride + (int64_t)(pos < 0 ? 0 : pos) * hidden;
    if (threadIdx.x == 0) {
        row_pos[row] = pos;
        row_src[row] = src;
        if (pos < 0) atomicOr(status, kFlagBadIndex);
    }
    rmsnorm_row(reinterpret_cast<const uint4*>(x + src), reinterpret_cast<const uint4*>(gain),
                reinterpret_cast<uint4*>(xn + (int64_t)row * hidden), hidden, eps, red);
}

__global__ void __launch_bounds__(256) rmsnorm_kernel(const __nv_bfloat16* __restrict__ x,
                                                      const __nv_bfloat16* __restrict__ gain, float eps,
                                                      int hidden, __nv_bfloat16* __restrict__ xn) {
    __shared__ float red[8];
    pdl_wait();
    pdl_launch_dependents();
    const int64_t row = blockIdx.x;
    rmsnorm_row(reinterpret_cast<const uint4*>(x + row * hidden), reinterpret_cast<const uint4*>(gain),
                reinterpret_cast<uint4*>(xn + row * hidden), hidden, eps, red);
}

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

void launch_gather_rmsnorm(const void* x, int x_is_compact, int64_t x_batch_stride, int hidden,
                           const int32_t* anchor_idx, int k, const int32_t* extra_rows, int e, int batch,
                           int affix_start, int affix_len, int ctx_len, const void* gain, float eps,
                           int32_t* row_pos, int64_t* row_src, void* xn, uint32_t* status, cudaStream_t stream) {
    const int n = batch * (k + e);
    if (n == 0) return;
    launch_pdl(gather_rmsnorm_kernel, n, 256, 0, stream,
        static_cast<const __nv_bfloat16*>(x), x_is_compact, x_batch_stride, hidden, anchor_idx, k, extra_rows, e,
        affix_start, affix_len, ctx_len, static_cast<const __nv_bfloat16*>(gain), eps, row_pos, row_src,
        static_cast<__nv_bfloat16*>(xn), status);
}

void launch_rmsnorm(const void* x, const void* gain, float eps, int n, int hidden, void* xn, cudaStream_t stream) {
    if (n == 0) return;
    launch_pdl(rmsnorm_kernel, n, 256, 0, stream, static_cast<const __nv_bfloat16*>(x),
                                          static_cast<const __nv_bfloat16*>(gain), eps, hidden,
                                          static_cast<__nv_bfloat16*>(xn));
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
