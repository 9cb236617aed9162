// Row helpers shared by the kernels of the selective recomputation (Section 3.3): where a
// compact row of the recompute set R = A u E sits in the context, and RMSNorm of one row.
#pragma once
#include "common.cuh"

namespace acache {

// Position of compact row i of request b (i < k: anchor relative to the affix start, else the
// (i-k)-th extra row); -1 if the stored index is out of range.
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

// Sum over the block in a fixed order (bitwise reproducible); red holds one float per warp.
__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < nw; ++i) t += red[i];
    __syncthreads();
    return t;
}

// out = bf16(x * rsqrt(mean(x^2) + eps) * g) for one row of `hidden` bf16 values; all threads
// of the block take part.  raw (optional): the row as it was read is stored there too.
__device__ __forceinline__ void rmsnorm_row(const uint4* __restrict__ xr, const uint4* __restrict__ g,
                                            uint4* __restrict__ out, int hidden, float eps, float* red,
                                            uint4* __restrict__ raw = nullptr) {
    const int nchunk = hidden >> 3;
    if (nchunk <= 3 * (int)blockDim.x) {
        // the row fits in three 16-byte pieces per thread: one pass, the row stays in registers, and the gain is
        // requested before the block-wide sum so that it arrives meanwhile
        uint4 u[3], gg[3];
        float ss1 = 0.f;
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const int c = threadIdx.x + i * blockDim.x;
            u[i] = c < nchunk ? __ldcg(xr + c) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const int c = threadIdx.x + i * blockDim.x;
            gg[i] = c < nchunk ? g[c] : make_uint4(0u, 0u, 0u, 0u);
        }
        if (raw) {
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const int c = threadIdx.x + i * blockDim.x;
                if (c < nchunk) raw[c] = u[i];
            }
        }
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) { const float a = bf16_lo(w[e]), b = bf16_hi(w[e]); ss1 += a * a + b * b; }
        }
        const float rstd1 = rsqrtf(block_sum(ss1, red) / (float)hidden + eps);
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const int c = threadIdx.x + i * blockDim.x;
            if (c < nchunk) {
                const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
                const uint32_t gw[4] = {gg[i].x, gg[i].y, gg[i].z, gg[i].w};
                uint32_t r[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    r[e] = pack_bf16(bf16_lo(w[e]) * rstd1 * bf16_lo(gw[e]), bf16_hi(w[e]) * rstd1 * bf16_hi(gw[e]));
                out[c] = make_uint4(r[0], r[1], r[2], r[3]);
            }
        }
        return;
    }
    float ss = 0.f;
    for (int c = threadIdx.x; c < nchunk; c += blockDim.x) {
        uint4 u = __ldcg(xr + c);
        if (raw) raw[c] = u;
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
        uint4 u = __ldcg(xr + c), gg = g[c];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
        const uint32_t gw[4] = {gg.x, gg.y, gg.z, gg.w};
        uint32_t r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            r[i] = pack_bf16(bf16_lo(w[i]) * rstd * bf16_lo(gw[i]), bf16_hi(w[i]) * rstd * bf16_hi(gw[i]));
        out[c] = make_uint4(r[0], r[1], r[2], r[3]);
    }
}

}  // namespace acache
