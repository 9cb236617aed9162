// Top-K anchor selection, Eq. 6: A = TopK({s_j}, K).  One CTA per request: an exact
// radix select on the fp32 bit pattern finds the K-th largest score, then one ordered
// pass over positions emits the anchors ascending, ties going to the lower position.
#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace acache {

constexpr int kTopkThreads = 1024;
constexpr int kTopkSmemKeys = 16384;   // keys cached in shared memory up to this L

// Order-preserving map fp32 -> uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t score_key(float f) {
    uint32_t u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;   // -0 and +0 compare equal
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive block scan of one int per thread (blockDim.x == kTopkThreads); returns the
// exclusive prefix and writes the block total to *total.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_tot[w] = inc;
    __syncthreads();
    if (w == 0) {
        int t = warp_tot[lane];
        int ti = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int u = __shfl_up_sync(0xffffffffu, ti, o);
            if (lane >= o) ti += u;
        }
        warp_tot[lane] = ti - t;          // exclusive warp offsets
        if (lane == 31) *total = ti;
    }
    __syncthreads();
    int r = warp_tot[w] + inc - v;
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(kTopkThreads) topk_kernel(float* scores, int L, int K,
                                                            int32_t* __restrict__ anchor_idx, int use_smem,
                                                            const float* __restrict__ head_partial, int n_heads,
                                                            int accumulate) {
    extern __shared__ uint32_t keys_s[];
    __shared__ int hist[256];
    __shared__ int warp_tot[32];
    __shared__ int s_total;
    __shared__ uint32_t s_prefix;
    __shared__ int s_want;

    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x;
    float* s = scores + (int64_t)b * L;
    int32_t* out = anchor_idx + (int64_t)b * K;
    const int tid = threadIdx.x;

    if (head_partial) {   // Eq. 5: ordered sum over heads, fused in front of the selection
        for (int j = tid; j < L; j += kTopkThreads) {
            float v = 0.f;
            const float* hp = head_partial + (int64_t)b * n_heads * L + j;
            int h = 0;
            for (; h + 32 <= n_heads; h += 32) {    // 32 loads in flight (one trip to L2), added in head order
                float t[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) t[i] = __ldcg(hp + (int64_t)(h + i) * L);
#pragma unroll
                for (int i = 0; i < 32; ++i) v += t[i];
            }
            for (; h + 8 <= n_heads; h += 8) {
                float t[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) t[i] = __ldcg(hp + (int64_t)(h + i) * L);
#pragma unroll
                for (int i = 0; i < 8; ++i) v += t[i];
            }
            for (; h < n_heads; ++h) v += __ldcg(hp + (int64_t)h * L);
            const float f = accumulate ? s[j] + v : v;
            s[j] = f;
            if (use_smem) keys_s[j] = score_key(f);          // the selection reads the keys from shared memory
        }
        __syncthreads();
    } else if (use_smem) {
        for (int j = tid; j < L; j += kTopkThreads) keys_s[j] = score_key(s[j]);
    }
    if (tid == 0) { s_prefix = 0u; s_want = K; }
    __syncthreads();
    auto key_at = [&](int j) -> uint32_t { return use_smem ? keys_s[j] : score_key(s[j]); };

    // radix select, most significant byte first: after the loop s_prefix is the key of the
    // K-th largest element and s_want the number of elements equal to it that are taken.
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        for (int j0 = 0; j0 < L; j0 += kTopkThreads) {
            // one shared-memory atomic per distinct digit per warp (scores often share their top bytes)
            const int j = j0 + tid;
            int digit = -1;
            if (j < L) {
                const uint32_t kk = key_at(j);
                if ((kk & mask) == prefix) digit = (kk >> shift) & 0xFF;
            }
            const unsigned peers = __match_any_sync(0xffffffffu, digit);
            if (digit >= 0 && (tid & 31) == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
        }
        __syncthreads();
        if (tid < 32) {
            // lane l owns digits 255-8l .. 248-8l (descending); find the digit where the running
            // count from the top reaches the wanted rank
            int cnt[8], mine = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { cnt[i] = hist[255 - 8 * tid - i]; mine += cnt[i]; }
            int inc = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_up_sync(0xffffffffu, inc, o);
                if (tid >= o) inc += t;
            }
            const int want = s_want;
            const int before = inc - mine;                 // elements in digits above this lane's
            if (before < want && want <= inc) {            // exactly one lane
                int w = want - before, d = 255 - 8 * tid;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (cnt[i] >= w) { d = 255 - 8 * tid - i; break; }
                    w -= cnt[i];
                }
                s_prefix = prefix | ((uint32_t)d << shift);
                s_want = w;
            }
        }
        __syncthreads();
    }
    const uint32_t tau = s_prefix;
    const int need_eq = s_want;

    // ordered compaction: position ascending, chunk by chunk
    int base_eq = 0, base_out = 0;
    for (int j0 = 0; j0 < L; j0 += kTopkThreads) {
        const int j = j0 + tid;
        uint32_t kk = j < L ? key_at(j) : 0u;
        const int is_gt = (j < L) && (kk > tau);
        const int is_eq = (j < L) && (kk == tau);
        int eq_rank = base_eq + block_exclusive_scan(is_eq, warp_tot, &s_total);
        const int eq_total = s_total;
        const int sel = is_gt || (is_eq && eq_rank < need_eq);
        int o = base_out + block_exclusive_scan(sel, warp_tot, &s_total);
        const int sel_total = s_total;
        if (sel && o < K) out[o] = j;
        base_eq += eq_total;
        base_out += sel_total;
    }
}

void launch_topk(float* scores, int batch, int affix_len, int k, int32_t* anchor_idx, const float* head_partial,
                 int n_heads, int accumulate, cudaStream_t stream) {
    if (batch == 0 || (k == 0 && !head_partial)) return;
    const int use_smem = affix_len <= kTopkSmemKeys;
    const size_t smem = use_smem ? (size_t)affix_len * sizeof(uint32_t) : 0;
    if (smem > 48 * 1024)
        cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kTopkSmemKeys * (int)sizeof(uint32_t));
    launch_pdl(topk_kernel, batch, kTopkThreads, smem, stream, scores, affix_len, k, anchor_idx, use_smem, head_partial,
               n_heads, accumulate);
}

}  // namespace acache
