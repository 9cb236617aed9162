// Anchor scoring, Eq. 4-5:  a[j,k,h] = Softmax_j(q_mask[k,h] . K_affix[j,kv(h)] / sqrt(d)),
// s_j (+)= sum_h sum_{k in M} a[j,k,h].
//
// Three kernels, no atomics on floats (bitwise reproducible):
//   1. row statistics: for every masked query row and head, the softmax max and
//      denominator over the normaliser's key range, split along the keys;
//   2. column sums: for every affix key and head, sum over the masked queries of
//      exp2(logit - max) / denominator (logits recomputed, K read a second time);
//   3. ordered sum over heads into scores.
// Logits run on the tensor cores (bf16 mma.sync, fp32 accumulate) so that the pass stays
// bound by the K_affix read, not by ALU work.
#include <cooperative_groups.h>

#include <atomic>

#include "../../include/acache.h"
#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace acache {

constexpr int kScoreSplit = 256;      // keys per CTA in the statistics pass
constexpr int kMaxMaskedSmem = 4096;  // masked rows whose statistics fit in shared memory

int score_num_splits(int norm_len) { return (norm_len + kScoreSplit - 1) / kScoreSplit; }

// Copy a [64 x D] bf16 tile (row stride `stride` elements) into swizzled shared memory:
// D/64 panels of [64 rows x 64 cols], each row 128 bytes.  Rows >= valid are zero-filled.
template <int D>
__device__ __forceinline__ void load_tile64(uint32_t smem_base, const __nv_bfloat16* g, int64_t stride, int valid,
                                            int tid, int nthreads) {
    constexpr int CPR = D / 8;   // 16-byte chunks per row
    for (int c = tid; c < 64 * CPR; c += nthreads) {
        int r = c / CPR, cc = c % CPR;
        int ok = r < valid;
        const __nv_bfloat16* src = g + (int64_t)(ok ? r : 0) * stride + cc * 8;
        cp_async16(smem_base + (cc >> 3) * 8192 + swz64(r, cc & 7), src, ok ? 16 : 0);
    }
}

// A fragments (16 rows x D) of this warp's rows [row0, row0+16) from a swizzled tile.
template <int D>
__device__ __forceinline__ void load_a_frags(uint32_t (&a)[D / 16][4], uint32_t smem_base, int row0, int lane) {
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        int r = row0 + (lane & 15);
        int chunk = ks * 2 + (lane >> 4);
        ldmatrix_x4(a[ks][0], a[ks][1], a[ks][2], a[ks][3], smem_base + (chunk >> 3) * 8192 + swz64(r, chunk & 7));
    }
}

// acc[nb][4] = A(16 x D) * B^T where B is a swizzled [64 x D] tile (rows = n index).
template <int D>
__device__ __forceinline__ void mma_16x64(float (&acc)[8][4], const uint32_t (&a)[D / 16][4], uint32_t smem_b,
                                          int lane) {
#pragma unroll
    for (int nb = 0; nb < 8; ++nb)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nb][i] = 0.f;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
        for (int np = 0; np < 4; ++np) {
            int n = np * 16 + (lane & 7) + ((lane >> 4) << 3);
            int chunk = ks * 2 + ((lane >> 3) & 1);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(b0, b1, b2, b3, smem_b + (chunk >> 3) * 8192 + swz64(n, chunk & 7));
            mma_bf16_16816(acc[np * 2], a[ks], b0, b1);
            mma_bf16_16816(acc[np * 2 + 1], a[ks], b2, b3);
        }
    }
}

// ---- pass 1: per-row softmax statistics over the normaliser's key range -------------------
template <int D>
__global__ void __launch_bounds__(128) score_stats_kernel(ScoreArgs a, int n_split, float scale_log2e) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int TILE = 64 * D * 2;
    const uint32_t sQ = smem_u32(smem), sK0 = sQ + TILE;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.y, h = blockIdx.x;     // heads fastest: CTAs running together read whole K rows
    const int mtiles = (a.m + 63) / 64;
    const int b = blockIdx.z / mtiles, mt = blockIdx.z % mtiles;
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int64_t qstride = (int64_t)a.n_heads * D, kstride = (int64_t)a.n_kv_heads * D;
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(a.q_mask) +
                             ((int64_t)b * a.m + mt * 64) * qstride + (int64_t)h * D;
    const int key_lo = split * kScoreSplit;
    const int key_n = min(kScoreSplit, a.norm_len - key_lo);
    const __nv_bfloat16* kbase = static_cast<const __nv_bfloat16*>(a.cache_k) + (int64_t)b * a.kv_batch_stride +
                                 (int64_t)(a.norm_lo + key_lo) * kstride + (int64_t)kvh * D;
    const int ntiles = (key_n + 63) / 64;

    // early_k: the cache was last written at least two kernels back (the layer-step: the masked rows' projection
    // sits in between), so the first key tile can be requested while the producer of Q is still running
    // all of the CTA's key tiles (at most kScoreSplit / 64 = 4) are requested at once: one trip to memory instead
    // of one per tile; with early_k (see ScoreArgs) before the wait for the producer of Q
    auto load_keys = [&]() {
        for (int t = 0; t < ntiles; ++t)
            load_tile64<D>(sK0 + t * TILE, kbase + (int64_t)t * 64 * kstride, kstride, min(64, key_n - t * 64), tid, 128);
    };
    if (a.early_k) load_keys();
    pdl_wait();
    pdl_launch_dependents();
    load_tile64<D>(sQ, q, qstride, min(64, a.m - mt * 64), tid, 128);
    if (!a.early_k) load_keys();
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();
    uint32_t af[D / 16][4];
    load_a_frags<D>(af, sQ, warp * 16, lane);

    float mx[2] = {-INFINITY, -INFINITY}, den[2] = {0.f, 0.f};
    for (int t = 0; t < ntiles; ++t) {
        const uint32_t sK = sK0 + t * TILE;
        float acc[8][4];
        mma_16x64<D>(acc, af, sK, lane);
        const int valid = key_n - t * 64;
        float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int col = nb * 8 + (lane & 3) * 2 + (i & 1);
                float s = col < valid ? acc[nb][i] * scale_log2e : -INFINITY;
                acc[nb][i] = s;
                tmax[i >> 1] = fmaxf(tmax[i >> 1], s);
            }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
            tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
            float nm = fmaxf(mx[r], tmax[r]);
            den[r] *= exp2f(mx[r] - nm);
            mx[r] = nm;
        }
        float part[2] = {0.f, 0.f};
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int i = 0; i < 4; ++i) part[i >> 1] += exp2f(acc[nb][i] - mx[i >> 1]);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            part[r] += __shfl_xor_sync(0xffffffffu, part[r], 1);
            part[r] += __shfl_xor_sync(0xffffffffu, part[r], 2);
            den[r] += part[r];
        }
    }
    if ((lane & 3) == 0) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            int row = mt * 64 + warp * 16 + (lane >> 2) + r * 8;
            if (row < a.m) {
                float* st = a.row_stats + ((((int64_t)b * a.n_heads + h) * n_split + split) * a.m + row) * 2;
                st[0] = mx[r];
                st[1] = den[r];
            }
        }
    }
}

// ---- pass 2: per-key column sums of the normalised weights -------------------------------
// One CTA = `kt_per_cta` consecutive tiles of 64 affix keys of one head (four when the masked rows fit
// one 64-row tile, so that the combination of the split statistics and the Q tile load are paid once
// per 256 keys; one otherwise, with the Q tiles streaming through a double buffer).
template <int D>
__global__ void __launch_bounds__(128) score_colsum_kernel(ScoreArgs a, int n_split, float scale_log2e, int kt_per_cta) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int TILE = 64 * D * 2;
    const uint32_t sK0 = smem_u32(smem), sQ0 = sK0 + 2 * TILE;
    float* s_max = reinterpret_cast<float*>(smem + 4 * TILE);
    float* s_inv = s_max + a.m;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = blockIdx.x, b = blockIdx.z;                     // heads fastest (see the statistics pass)
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int64_t qstride = (int64_t)a.n_heads * D, kstride = (int64_t)a.n_kv_heads * D;
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(a.q_mask) + (int64_t)b * a.m * qstride + (int64_t)h * D;
    const int key_tiles = (a.affix_len + 63) / 64;
    const int jt_first = blockIdx.y * kt_per_cta;
    const int n_my = min(kt_per_cta, key_tiles - jt_first);
    const __nv_bfloat16* kbase = static_cast<const __nv_bfloat16*>(a.cache_k) + (int64_t)b * a.kv_batch_stride +
                                 (int64_t)a.affix_start * kstride + (int64_t)kvh * D;
    const int mtiles = (a.m + 63) / 64;

    if (a.early_k)
        load_tile64<D>(sK0, kbase + (int64_t)jt_first * 64 * kstride, kstride, min(64, a.affix_len - jt_first * 64), tid, 128);
    pdl_wait();
    pdl_launch_dependents();
    if (!a.early_k)
        load_tile64<D>(sK0, kbase + (int64_t)jt_first * 64 * kstride, kstride, min(64, a.affix_len - jt_first * 64), tid, 128);
    load_tile64<D>(sQ0, q, qstride, min(64, a.m), tid, 128);
    cp_async_commit();

    // combine the split statistics of every masked row (fixed order)
    const float* st = a.row_stats + ((int64_t)b * a.n_heads + h) * n_split * a.m * 2;
    for (int r = tid; r < a.m; r += 128) {
        float M = -INFINITY;
        for (int s = 0; s < n_split; ++s) M = fmaxf(M, st[((int64_t)s * a.m + r) * 2]);
        float Dn = 0.f;
        for (int s = 0; s < n_split; ++s)
            Dn += st[((int64_t)s * a.m + r) * 2 + 1] * exp2f(st[((int64_t)s * a.m + r) * 2] - M);
        s_max[r] = M;
        s_inv[r] = 1.f / Dn;
    }
    for (int kt = 0; kt < n_my; ++kt) {
        const int j0 = (jt_first + kt) * 64;
        cp_async_wait<0>();
        __syncthreads();
        if (kt + 1 < n_my) {
            load_tile64<D>(sK0 + ((kt + 1) & 1) * TILE, kbase + (int64_t)(j0 + 64) * kstride, kstride,
                           min(64, a.affix_len - (j0 + 64)), tid, 128);
            cp_async_commit();
        }
        uint32_t af[D / 16][4];
        load_a_frags<D>(af, sK0 + (kt & 1) * TILE, warp * 16, lane);

        float colsum[2] = {0.f, 0.f};
        for (int t = 0; t < mtiles; ++t) {
            const uint32_t sQ = sQ0 + (t & 1) * TILE;
            if (t + 1 < mtiles) {          // only with one key tile per CTA: nothing else is in flight
                load_tile64<D>(sQ0 + ((t + 1) & 1) * TILE, q + (int64_t)(t + 1) * 64 * qstride, qstride,
                               min(64, a.m - (t + 1) * 64), tid, 128);
                cp_async_commit();
            }
            float acc[8][4];
            mma_16x64<D>(acc, af, sQ, lane);   // rows = keys, cols = masked queries
#pragma unroll
            for (int nb = 0; nb < 8; ++nb)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    int qrow = t * 64 + nb * 8 + (lane & 3) * 2 + (i & 1);
                    if (qrow < a.m) colsum[i >> 1] += exp2f(acc[nb][i] * scale_log2e - s_max[qrow]) * s_inv[qrow];
                }
            if (t + 1 < mtiles) {
                cp_async_wait<0>();
                __syncthreads();
            }
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            colsum[r] += __shfl_xor_sync(0xffffffffu, colsum[r], 1);
            colsum[r] += __shfl_xor_sync(0xffffffffu, colsum[r], 2);
        }
        if ((lane & 3) == 0) {
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                int j = j0 + warp * 16 + (lane >> 2) + r * 8;
                if (j < a.affix_len) a.head_partial[((int64_t)b * a.n_heads + h) * a.affix_len + j] = colsum[r];
            }
        }
    }
}

// ---- both passes in one launch: short affixes, one request or a few ----------------------------------
// With at most 1024 affix keys a head's work is cut over a cluster of eight CTAs, 64 or 128 keys each: every CTA takes
// the softmax statistics of all masked rows over its own keys, the four parts meet through distributed shared
// memory, and each CTA then takes the column sums of its own keys from the tiles it already holds.  One launch
// instead of two, and the statistics never leave the cluster.  Only when the normaliser runs over the affix
// keys themselves and the grid fits the SMs in one wave.
constexpr int kSmallCluster = 8;

template <int D, int kSmallTiles>          // key tiles per CTA: 1 (up to 512 affix keys) or 2 (up to 1024)
__global__ void __cluster_dims__(kSmallCluster, 1, 1) __launch_bounds__(128) score_small_kernel(ScoreArgs a, float scale_log2e) {
    namespace cg = cooperative_groups;
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int TILE = 64 * D * 2;
    const uint32_t sQ = smem_u32(smem), sK0 = sQ + TILE;
    float* s_stat = reinterpret_cast<float*>(smem + (1 + kSmallTiles) * TILE);     // [tile][64 rows][max, den]
    float* s_max = s_stat + kSmallTiles * 128;
    float* s_inv = s_max + 64;
    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = blockIdx.x % kSmallCluster, h = blockIdx.x / kSmallCluster, b = blockIdx.y;
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int64_t qstride = (int64_t)a.n_heads * D, kstride = (int64_t)a.n_kv_heads * D;
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(a.q_mask) + (int64_t)b * a.m * qstride + (int64_t)h * D;
    const int key0 = rank * kSmallTiles * 64;                                      // first affix key of this CTA
    const __nv_bfloat16* kbase = static_cast<const __nv_bfloat16*>(a.cache_k) + (int64_t)b * a.kv_batch_stride +
                                 (int64_t)(a.affix_start + key0) * kstride + (int64_t)kvh * D;
    const int nkeys = max(0, min(kSmallTiles * 64, a.affix_len - key0));
    const int ntiles = (nkeys + 63) / 64;
    auto load_keys = [&]() {
        for (int t = 0; t < ntiles; ++t)
            load_tile64<D>(sK0 + t * TILE, kbase + (int64_t)t * 64 * kstride, kstride, min(64, nkeys - t * 64), tid, 128);
    };
    if (a.early_k) load_keys();          // see ScoreArgs::early_k
    pdl_wait();
    pdl_launch_dependents();
    load_tile64<D>(sQ, q, qstride, min(64, a.m), tid, 128);
    if (!a.early_k) load_keys();
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();

    // pass 1: warp w takes the 16-row group (w & 1) [+ 2 in a second round] over key tile w >> 1
    const int groups = (a.m + 15) / 16;
    constexpr int WPT = 4 / kSmallTiles;      // warps per key tile
    for (int g0 = 0; g0 < groups; g0 += WPT) {
        const int rg = g0 + warp % WPT, t = warp / WPT;
        if (rg >= groups) continue;
        float mx[2] = {-INFINITY, -INFINITY}, den[2] = {0.f, 0.f};
        if (t < ntiles) {
            uint32_t af[D / 16][4];
            load_a_frags<D>(af, sQ, rg * 16, lane);
            float acc[8][4];
            mma_16x64<D>(acc, af, sK0 + t * TILE, lane);
            const int valid = nkeys - t * 64;
#pragma unroll
            for (int nb = 0; nb < 8; ++nb)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int col = nb * 8 + (lane & 3) * 2 + (i & 1);
                    const float sc = col < valid ? acc[nb][i] * scale_log2e : -INFINITY;
                    acc[nb][i] = sc;
                    mx[i >> 1] = fmaxf(mx[i >> 1], sc);
                }
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            }
#pragma unroll
            for (int nb = 0; nb < 8; ++nb)
#pragma unroll
                for (int i = 0; i < 4; ++i) den[i >> 1] += exp2f(acc[nb][i] - mx[i >> 1]);
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                den[r] += __shfl_xor_sync(0xffffffffu, den[r], 1);
                den[r] += __shfl_xor_sync(0xffffffffu, den[r], 2);
            }
        }
        if ((lane & 3) == 0) {
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int row = rg * 16 + (lane >> 2) + r * 8;
                s_stat[(t * 64 + row) * 2] = mx[r];
                s_stat[(t * 64 + row) * 2 + 1] = den[r];
            }
        }
    }
    cluster.sync();
    if (tid < groups * 16) {
        float ms[kSmallCluster * kSmallTiles], ds[kSmallCluster * kSmallTiles];
#pragma unroll
        for (int c = 0; c < kSmallCluster; ++c) {
            const float* remote = cluster.map_shared_rank(s_stat, c);
#pragma unroll
            for (int t = 0; t < kSmallTiles; ++t) {
                const float2 v = *reinterpret_cast<const float2*>(remote + (t * 64 + tid) * 2);
                ms[c * kSmallTiles + t] = v.x;
                ds[c * kSmallTiles + t] = v.y;
            }
        }
        float M = -INFINITY, Dn = 0.f;
#pragma unroll
        for (int i = 0; i < kSmallCluster * kSmallTiles; ++i) M = fmaxf(M, ms[i]);
#pragma unroll
        for (int i = 0; i < kSmallCluster * kSmallTiles; ++i)
            if (ms[i] != -INFINITY) Dn += ds[i] * exp2f(ms[i] - M);
        s_max[tid] = M;
        s_inv[tid] = 1.f / Dn;
    }
    __syncthreads();

    // pass 2: column sums of the normalised weights over this CTA's keys, 16 keys of every tile per warp
    for (int kt = 0; kt < ntiles; ++kt) {
        uint32_t af[D / 16][4];
        load_a_frags<D>(af, sK0 + kt * TILE, warp * 16, lane);
        float acc[8][4];
        mma_16x64<D>(acc, af, sQ, lane);       // rows = keys, cols = masked queries
        float colsum[2] = {0.f, 0.f};
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int qrow = nb * 8 + (lane & 3) * 2 + (i & 1);
                if (qrow < a.m) colsum[i >> 1] += exp2f(acc[nb][i] * scale_log2e - s_max[qrow]) * s_inv[qrow];
            }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            colsum[r] += __shfl_xor_sync(0xffffffffu, colsum[r], 1);
            colsum[r] += __shfl_xor_sync(0xffffffffu, colsum[r], 2);
        }
        if ((lane & 3) == 0) {
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int j = key0 + kt * 64 + warp * 16 + (lane >> 2) + r * 8;
                if (j < a.affix_len) a.head_partial[((int64_t)b * a.n_heads + h) * a.affix_len + j] = colsum[r];
            }
        }
    }
    cluster.sync();        // no CTA leaves while a neighbour may still read its statistics
}

// ---- pass 3: ordered sum over heads -------------------------------------------------------
__global__ void __launch_bounds__(256) score_reduce_heads_kernel(const float* __restrict__ head_partial,
                                                                 float* __restrict__ scores, int n_heads, int L,
                                                                 int accumulate) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= L) return;
    float s = 0.f;
    for (int h = 0; h < n_heads; ++h) s += head_partial[((int64_t)b * n_heads + h) * L + j];
    float* out = scores + (int64_t)b * L + j;
    *out = accumulate ? *out + s : s;
}

template <int D>
static int launch_score_d(const ScoreArgs& a, cudaStream_t stream) {
    const int n_split = score_num_splits(a.norm_len);
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)D);
    constexpr int TILE = 64 * D * 2;
    const int mtiles = (a.m + 63) / 64;
    const size_t smem1 = (1 + kScoreSplit / 64) * TILE;      // the Q tile and all of a split's key tiles
    const size_t smem2 = 4 * TILE + (size_t)a.m * 8;
    const int key_tiles = (a.affix_len + 63) / 64;
    // several key tiles per CTA only while that still leaves a few waves of CTAs (measured: L = 512, B = 1 is
    // faster with one tile per CTA, L = 8192 with four)
    const int64_t ctas1 = (int64_t)a.n_heads * key_tiles * a.batch;
    const int kt_per_cta = mtiles > 1 ? 1 : ctas1 >= 2400 ? 4 : ctas1 >= 1200 ? 2 : 1;
    static const bool small_on = [] { const char* e = getenv("ACACHE_SCORE_SMALL"); return !e || atoi(e) != 0; }();
    if (small_on && a.norm_lo == a.affix_start && a.norm_len == a.affix_len && a.affix_len <= 128 * kSmallCluster && a.m <= 64 &&
        a.n_heads * a.batch <= 148) {
        const int tpc = a.affix_len <= 64 * kSmallCluster ? 1 : 2;
        const size_t smem0 = (size_t)(1 + tpc) * TILE + (tpc * 128 + 128) * sizeof(float);
        auto kernel = tpc == 1 ? score_small_kernel<D, 1> : score_small_kernel<D, 2>;
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem0);
        launch_pdl(kernel, dim3(a.n_heads * kSmallCluster, a.batch), 128, smem0, stream, a, scale_log2e);
        if (a.defer_head_sum) return 1;
        launch_pdl(score_reduce_heads_kernel, dim3((a.affix_len + 255) / 256, a.batch), 256, 0, stream, a.head_partial,
                   a.scores, a.n_heads, a.affix_len, a.accumulate);
        return 2;
    }
    cudaFuncSetAttribute(score_stats_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
    cudaFuncSetAttribute(score_colsum_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
    launch_pdl(score_stats_kernel<D>, dim3(a.n_heads, n_split, a.batch * mtiles), 128, smem1, stream, a, n_split,
               scale_log2e);
    launch_pdl(score_colsum_kernel<D>, dim3(a.n_heads, (key_tiles + kt_per_cta - 1) / kt_per_cta, a.batch), 128, smem2, stream, a,
               n_split, scale_log2e, kt_per_cta);
    if (a.defer_head_sum) return 2;   // the selection kernel sums the heads itself
    launch_pdl(score_reduce_heads_kernel, dim3((a.affix_len + 255) / 256, a.batch), 256, 0, stream, a.head_partial,
               a.scores, a.n_heads, a.affix_len, a.accumulate);
    return 3;
}

int launch_score(const ScoreArgs& a, cudaStream_t stream) {
    if (a.batch == 0 || a.affix_len == 0) return 0;
    if (a.m == 0) {   // no masked rows: this layer contributes nothing
        if (!a.accumulate) cudaMemsetAsync(a.scores, 0, (size_t)a.batch * a.affix_len * sizeof(float), stream);
        return 0;
    }
    if (a.m > kMaxMaskedSmem) return -1;
    const int tc = launch_score_tc(a, a.status, stream);
    if (tc < 0) return -1;
    if (tc > 0) {
        if (a.defer_head_sum) return tc;
        launch_pdl(score_reduce_heads_kernel, dim3((a.affix_len + 255) / 256, a.batch), 256, 0, stream, a.head_partial,
                   a.scores, a.n_heads, a.affix_len, a.accumulate);
        return tc + 1;
    }
    return a.head_dim == 128 ? launch_score_d<128>(a, stream) : launch_score_d<64>(a, stream);
}

}  // namespace acache

// ---- scoring without any allocation ------------------------------------------------------------
// Scratch of the allocation-free entry point: lives in the library's device image, so every
// GPU that loads the library holds these 4 MiB until the process exits.
#define ACACHE_STATIC_SCRATCH_FLOATS (1u << 20)
static __device__ __align__(256) float g_static_score_scratch[ACACHE_STATIC_SCRATCH_FLOATS];

namespace {
constexpr int kMaxDevices = 64;
// device address of the array, per device; atomic, so that first calls from two host threads are safe (both
// look the same address up)
std::atomic<float*> g_static_scratch_ptr[kMaxDevices];
}  // namespace

extern "C" acache_status acache_score_anchors_static(const acache_model_desc* shape, const acache_request* req,
                                                     const void* q_mask, const acache_kv* kv, float* scores,
                                                     int accumulate, int norm_full, acache_stream_t stream) {
    using namespace acache;
    if (!shape || !req || !kv || !scores) return ACACHE_ERR_INVALID_ARG;
    if ((shape->head_dim != 64 && shape->head_dim != 128) || shape->n_heads <= 0 || shape->n_kv_heads <= 0 ||
        shape->n_heads % shape->n_kv_heads)
        return ACACHE_ERR_UNSUPPORTED_SHAPE;
    if (req->batch < 0 || req->ctx_len <= 0 || req->affix_len < 0 || req->affix_start < 0 || req->n_masked < 0 ||
        (int64_t)req->affix_start + req->affix_len > req->ctx_len)
        return ACACHE_ERR_INVALID_ARG;
    // batch_stride 0: one cache shared by every request of the batch (Section 4.1), as in acache_score_anchors
    if (!kv->k || (reinterpret_cast<uintptr_t>(kv->k) & 15u) || kv->ctx_capacity < req->ctx_len ||
        (kv->batch_stride != 0 &&
         (kv->batch_stride < (int64_t)kv->ctx_capacity * shape->n_kv_heads * shape->head_dim || (kv->batch_stride & 7))))
        return ACACHE_ERR_INVALID_ARG;
    if (req->n_masked > 0 && (!q_mask || (reinterpret_cast<uintptr_t>(q_mask) & 15u))) return ACACHE_ERR_INVALID_ARG;
    if (req->n_masked > kMaxMaskedSmem) return ACACHE_ERR_UNSUPPORTED_SHAPE;

    const int norm_len = norm_full ? req->ctx_len : req->affix_len;
    const uint64_t stats_floats = (uint64_t)req->batch * shape->n_heads * score_num_splits(norm_len) * req->n_masked * 2;
    const uint64_t partial_floats = (uint64_t)req->batch * shape->n_heads * req->affix_len;
    const uint64_t stats_padded = (stats_floats + 63) & ~uint64_t(63);
    if (stats_padded + partial_floats > ACACHE_STATIC_SCRATCH_FLOATS) return ACACHE_ERR_WORKSPACE;

    // Set-up, once per device, with that device current: the array's name is only a host-side
    // handle here, so ask the runtime for the address the kernels must be given.
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ACACHE_ERR_CUDA;
    float* scratch = g_static_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&scratch), g_static_score_scratch) != cudaSuccess || !scratch) {
            (void)cudaGetLastError();
            return ACACHE_ERR_CUDA;
        }
        g_static_scratch_ptr[dev].store(scratch, std::memory_order_release);
    }

    ScoreArgs a{};
    a.q_mask = q_mask;
    a.cache_k = kv->k;
    a.kv_batch_stride = kv->batch_stride;
    a.batch = req->batch; a.m = req->n_masked;
    a.n_heads = shape->n_heads; a.n_kv_heads = shape->n_kv_heads; a.head_dim = shape->head_dim;
    a.affix_start = req->affix_start; a.affix_len = req->affix_len;
    a.norm_lo = norm_full ? 0 : req->affix_start;
    a.norm_len = norm_len;
    a.row_stats = scratch;                    // every word the kernels read is written earlier in the same call,
    a.head_partial = scratch + stats_padded;  // so nothing needs clearing between calls
    a.scores = scores;
    a.accumulate = accumulate;
    a.defer_head_sum = 0;
    if (launch_score(a, stream) < 0) return ACACHE_ERR_UNSUPPORTED_SHAPE;
    return cudaGetLastError() == cudaSuccess ? ACACHE_OK : ACACHE_ERR_CUDA;
}

