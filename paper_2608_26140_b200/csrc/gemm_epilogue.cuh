// Epilogues of the projection GEMMs, shared by every GEMM main loop.  The main loop leaves
// its fp32 accumulator tile [128 rows x 128 cols] in shared memory (row pitch kStagePitch
// floats); the functions below turn it into the bf16 tensors the path stores.
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace acache {

constexpr int kStagePitch = 132;   // floats per staged row (128 + 4 padding)

__device__ __forceinline__ uint4 pack8(const float* v) {
    return make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}

// q/k/v projection: bias, rotary embedding with the rotate-half pairing (i, i + d/2) at the
// row's absolute position, bf16 store to the compact output and, for k/v, optionally straight
// into the cache row the fresh state belongs to (scatter fused: store-then-attend).
__device__ __forceinline__ void epilogue_qkv(const GemmArgs& g, const float* stage, int m0, int seg, int c0,
                                             int tid, int nthreads) {
    const int d = g.head_dim, half = d >> 1;
    const int heads_in_tile = 128 / d;
    const int chunks = half >> 3;                       // 8-wide chunks per half head
    const int items = 128 * heads_in_tile * chunks;
    const int nseg = g.n[seg];
    const bool do_rope = seg < g.rope_segments;
    const __nv_bfloat16* bias = static_cast<const __nv_bfloat16*>(g.bias[seg]);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(g.out[seg]);
    __nv_bfloat16* cache = seg == 1 ? static_cast<__nv_bfloat16*>(g.cache_k)
                         : seg == 2 ? static_cast<__nv_bfloat16*>(g.cache_v) : nullptr;
    for (int it = tid; it < items; it += nthreads) {
        const int ch = it % chunks;
        const int hd = (it / chunks) % heads_in_tile;
        const int r = it / (chunks * heads_in_tile);
        const int row = m0 + r;
        if (row >= g.M) continue;
        const int pos = g.row_pos[row];
        const int cl = hd * d + ch * 8;                 // tile column of the low half
        float lo[8], hi[8];
        const float* sp = stage + r * kStagePitch + cl;
#pragma unroll
        for (int i = 0; i < 8; ++i) { lo[i] = sp[i]; hi[i] = sp[half + i]; }
        if (bias) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                lo[i] += __bfloat162float(bias[c0 + cl + i]);
                hi[i] += __bfloat162float(bias[c0 + cl + half + i]);
            }
        }
        if (do_rope) {
            const int p = pos < 0 ? 0 : pos;
            const float4* cs = reinterpret_cast<const float4*>(g.rope_cos + (int64_t)p * half + ch * 8);
            const float4* sn = reinterpret_cast<const float4*>(g.rope_sin + (int64_t)p * half + ch * 8);
            float4 c0v = cs[0], c1v = cs[1], s0v = sn[0], s1v = sn[1];
            const float c[8] = {c0v.x, c0v.y, c0v.z, c0v.w, c1v.x, c1v.y, c1v.z, c1v.w};
            const float s[8] = {s0v.x, s0v.y, s0v.z, s0v.w, s1v.x, s1v.y, s1v.z, s1v.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float a = lo[i], b = hi[i];
                lo[i] = a * c[i] - b * s[i];
                hi[i] = b * c[i] + a * s[i];
            }
        }
        const uint4 plo = pack8(lo), phi = pack8(hi);
        if (out) {
            __nv_bfloat16* o = out + (int64_t)row * nseg + c0 + cl;
            *reinterpret_cast<uint4*>(o) = plo;
            *reinterpret_cast<uint4*>(o + half) = phi;
        }
        if (cache && pos >= 0) {
            const int b = row / g.rows_per_req;
            __nv_bfloat16* o = cache + (int64_t)b * g.kv_batch_stride + (int64_t)pos * nseg + c0 + cl;
            *reinterpret_cast<uint4*>(o) = plo;
            *reinterpret_cast<uint4*>(o + half) = phi;
        }
    }
}

// out[row, n0 + c] = bf16(resid[row] + acc)
__device__ __forceinline__ void epilogue_residual(const GemmArgs& g, const float* stage, int m0, int n0, int N,
                                                  int tid, int nthreads) {
    const __nv_bfloat16* resid = static_cast<const __nv_bfloat16*>(g.resid);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(g.c);
    for (int it = tid; it < 128 * 16; it += nthreads) {
        const int r = it >> 4, ch = it & 15;
        const int row = m0 + r;
        if (row >= g.M) continue;
        const int64_t roff = g.resid_off ? g.resid_off[row] : (int64_t)row * N;
        const uint4 rv = *reinterpret_cast<const uint4*>(resid + roff + n0 + ch * 8);
        const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
        const float* sp = stage + r * kStagePitch + ch * 8;
        float v[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = sp[2 * i] + bf16_lo(rw[i]);
            v[2 * i + 1] = sp[2 * i + 1] + bf16_hi(rw[i]);
        }
        *reinterpret_cast<uint4*>(out + (int64_t)row * N + n0 + ch * 8) = pack8(v);
    }
}

// Tile columns 0..63 are gate, 64..127 are up, both for MLP columns [f0, f0 + 64):
// out[row, f0 + c] = bf16(silu(gate) * up)
__device__ __forceinline__ void epilogue_swiglu(const GemmArgs& g, const float* stage, int m0, int f0, int Fm,
                                                int tid, int nthreads) {
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(g.c);
    for (int it = tid; it < 128 * 8; it += nthreads) {
        const int r = it >> 3, ch = it & 7;
        const int row = m0 + r;
        if (row >= g.M) continue;
        const float* sp = stage + r * kStagePitch + ch * 8;
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float gt = sp[i], up = sp[64 + i];
            v[i] = gt / (1.f + __expf(-gt)) * up;
        }
        *reinterpret_cast<uint4*>(out + (int64_t)row * Fm + f0 + ch * 8) = pack8(v);
    }
}

}  // namespace acache
