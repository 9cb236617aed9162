// Bidirectional attention of the recomputed rows over the whole logical context
// (Section 4.3: queries only for R, keys/values for all T positions, no mask).
// Online-softmax tiles: S = Q K^T and O += P V on bf16 tensor-core tiles with fp32
// accumulation and fp32 softmax statistics.  Keys/values come from the token-major cache or,
// where a position -> fresh-row map says so, from the compact fresh K/V (the logical view of
// the working cache without having written it).  This file holds the mma.sync kernels (head
// dimension 64, and the fallback when the tcgen05 kernel of attn_tc.cu is switched off) and
// the dispatch between the two.
#include <cstdlib>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"

namespace acache {

constexpr int kAttnTargetCtas = 296;   // two CTAs per SM on 148 SMs

template <int D>
__device__ __forceinline__ void load_q_tile(uint32_t sdst, const __nv_bfloat16* q, int64_t stride, int valid, int tid) {
    constexpr int CPR = D / 8;
    for (int c = tid; c < 64 * CPR; c += 128) {
        int r = c / CPR, cc = c % CPR;
        int ok = r < valid;
        cp_async16(sdst + (cc >> 3) * 8192 + swz64(r, cc & 7), q + (int64_t)(ok ? r : 0) * stride + cc * 8, ok ? 16 : 0);
    }
}

template <int D>
__device__ __forceinline__ void load_kv_tile(uint32_t sk, uint32_t sv, const AttnArgs& a, int b, int kvh, int t0,
                                             int tid) {
    constexpr int CPR = D / 8;
    const int64_t kstride = (int64_t)a.n_kv_heads * D;
    const __nv_bfloat16* ck = static_cast<const __nv_bfloat16*>(a.cache_k) + (int64_t)b * a.kv_batch_stride + kvh * D;
    const __nv_bfloat16* cv = static_cast<const __nv_bfloat16*>(a.cache_v) + (int64_t)b * a.kv_batch_stride + kvh * D;
    const int n_fresh = a.n_fresh ? a.n_fresh : a.n;
    const __nv_bfloat16* nk = static_cast<const __nv_bfloat16*>(a.k_new) + (int64_t)b * n_fresh * kstride + kvh * D;
    const __nv_bfloat16* nv = static_cast<const __nv_bfloat16*>(a.v_new) + (int64_t)b * n_fresh * kstride + kvh * D;
    for (int c = tid; c < 64 * CPR; c += 128) {
        int r = c / CPR, cc = c % CPR;
        int t = t0 + r;
        int ok = t < a.ctx_len;
        const __nv_bfloat16 *pk, *pv;
        int s = (ok && a.slot) ? a.slot[(int64_t)b * a.ctx_len + t] : -1;
        if (s >= 0) {
            pk = nk + (int64_t)s * kstride;
            pv = nv + (int64_t)s * kstride;
        } else {
            pk = ck + (int64_t)(ok ? t : 0) * kstride;
            pv = cv + (int64_t)(ok ? t : 0) * kstride;
        }
        uint32_t off = (cc >> 3) * 8192 + swz64(r, cc & 7);
        cp_async16(sk + off, pk + cc * 8, ok ? 16 : 0);
        cp_async16(sv + off, pv + cc * 8, ok ? 16 : 0);
    }
}

constexpr int ATT_STAGES = 3;

// One CTA: 64 query rows of one head against the key tiles [tile_lo, tile_hi) of its split.
// With one split the normalised output is written directly; otherwise the unnormalised fp32
// accumulator and the row statistics go to scratch and attention_combine_kernel merges them.
template <int D>
__global__ void __launch_bounds__(128) attention_kernel(const AttnArgs a, float scale_log2e, int n_split,
                                                        int tiles_per_split) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int TILE = 64 * D * 2;
    const uint32_t sQ = smem_u32(smem);
    pdl_wait();
    pdl_launch_dependents();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int qt = blockIdx.x / n_split, split = blockIdx.x % n_split, h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int64_t qstride = (int64_t)a.n_heads * D;
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(a.q) + ((int64_t)b * a.n + qt * 64) * qstride + h * D;
    const int all_tiles = (a.ctx_len + 63) / 64;
    const int tile_lo = split * tiles_per_split;
    const int ntiles = min(all_tiles, tile_lo + tiles_per_split) - tile_lo;
    auto sK = [&](int buf) { return sQ + TILE + buf * 2 * TILE; };
    auto sV = [&](int buf) { return sQ + 2 * TILE + buf * 2 * TILE; };

    load_q_tile<D>(sQ, q, qstride, min(64, a.n - qt * 64), tid);
    load_kv_tile<D>(sK(0), sV(0), a, b, kvh, tile_lo * 64, tid);
    cp_async_commit();
    if (ntiles > 1) load_kv_tile<D>(sK(1), sV(1), a, b, kvh, (tile_lo + 1) * 64, tid);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();

    uint32_t qf[D / 16][4];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        int r = warp * 16 + (lane & 15);
        int chunk = ks * 2 + (lane >> 4);
        ldmatrix_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], sQ + (chunk >> 3) * 8192 + swz64(r, chunk & 7));
    }

    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
    float mx[2] = {-INFINITY, -INFINITY}, den[2] = {0.f, 0.f};

    for (int t = 0; t < ntiles; ++t) {
        // tile t is resident (waited for below); prefetch tile t + 2 into the buffer tile t - 1 used
        if (t + 2 < ntiles) load_kv_tile<D>(sK((t + 2) % ATT_STAGES), sV((t + 2) % ATT_STAGES), a, b, kvh,
                                            (tile_lo + t + 2) * 64, tid);
        cp_async_commit();
        const uint32_t sk = sK(t % ATT_STAGES), sv = sV(t % ATT_STAGES);
        float s[8][4];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int i = 0; i < 4; ++i) s[nb][i] = 0.f;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                int n = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                int chunk = ks * 2 + ((lane >> 3) & 1);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3, sk + (chunk >> 3) * 8192 + swz64(n, chunk & 7));
                mma_bf16_16816(s[np * 2], qf[ks], b0, b1);
                mma_bf16_16816(s[np * 2 + 1], qf[ks], b2, b3);
            }
        }
        const int valid = a.ctx_len - (tile_lo + t) * 64;
        // keys that do not exist (DropNA layout): two mask words per 64-key tile
        uint32_t drop[2] = {0u, 0u};
        if (a.key_drop) {
            const int w0 = (tile_lo + t) * 2;
            const uint32_t* kd = a.key_drop + (int64_t)b * a.excl_words;
            if (w0 < a.excl_words) drop[0] = __ldg(kd + w0);
            if (w0 + 1 < a.excl_words) drop[1] = __ldg(kd + w0 + 1);
        }
        float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int col = nb * 8 + (lane & 3) * 2 + (i & 1);
                const bool there = col < valid && !((drop[col >> 5] >> (col & 31)) & 1u);
                float v = there ? s[nb][i] * scale_log2e : -INFINITY;
                s[nb][i] = v;
                tmax[i >> 1] = fmaxf(tmax[i >> 1], v);
            }
        float corr[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
            tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
            float nm = fmaxf(mx[r], tmax[r]);
            corr[r] = nm == -INFINITY ? 1.f : exp2f(mx[r] - nm);      // no key seen yet (a tile may be dropped whole)
            mx[r] = nm;
            den[r] *= corr[r];
        }
        const float mref[2] = {mx[0] == -INFINITY ? 0.f : mx[0], mx[1] == -INFINITY ? 0.f : mx[1]};
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            o[i][0] *= corr[0]; o[i][1] *= corr[0];
            o[i][2] *= corr[1]; o[i][3] *= corr[1];
        }
        uint32_t pf[4][4];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            float p0 = exp2f(s[nb][0] - mref[0]), p1 = exp2f(s[nb][1] - mref[0]);
            float p2 = exp2f(s[nb][2] - mref[1]), p3 = exp2f(s[nb][3] - mref[1]);
            den[0] += p0 + p1;
            den[1] += p2 + p3;
            pf[nb >> 1][(nb & 1) * 2] = pack_bf16(p0, p1);
            pf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int np = 0; np < D / 16; ++np) {
                int key = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                int chunk = np * 2 + (lane >> 4);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(b0, b1, b2, b3, sv + (chunk >> 3) * 8192 + swz64(key, chunk & 7));
                mma_bf16_16816(o[np * 2], pf[kk], b0, b1);
                mma_bf16_16816(o[np * 2 + 1], pf[kk], b2, b3);
            }
        }
        cp_async_wait<1>();     // everything but the newest group: tile t + 1 has landed
        __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        den[r] += __shfl_xor_sync(0xffffffffu, den[r], 1);
        den[r] += __shfl_xor_sync(0xffffffffu, den[r], 2);
    }
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(a.o);
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = qt * 64 + warp * 16 + (lane >> 2) + r * 8;
        if (row >= a.n) continue;
        if (n_split == 1) {
            const float inv = 1.f / den[r];
            __nv_bfloat16* orow = out + ((int64_t)b * a.n + row) * qstride + h * D;
#pragma unroll
            for (int nb = 0; nb < D / 8; ++nb) {
                int col = nb * 8 + (lane & 3) * 2;
                *reinterpret_cast<uint32_t*>(orow + col) = pack_bf16(o[nb][r * 2] * inv, o[nb][r * 2 + 1] * inv);
            }
        } else {
            const int64_t rh = ((int64_t)b * a.n + row) * a.n_heads + h;
            float* po = a.part_o + (rh * n_split + split) * D;
#pragma unroll
            for (int nb = 0; nb < D / 8; ++nb) {
                int col = nb * 8 + (lane & 3) * 2;
                *reinterpret_cast<float2*>(po + col) = make_float2(o[nb][r * 2], o[nb][r * 2 + 1]);
            }
            if ((lane & 3) == 0) {
                a.part_ml[(rh * n_split + split) * 2] = mx[r];
                a.part_ml[(rh * n_split + split) * 2 + 1] = den[r];
            }
        }
    }
}

// Merges the key splits of one (row, head): o = sum_s O_s 2^(m_s - m) / sum_s l_s 2^(m_s - m).
template <int D>
__global__ void __launch_bounds__(128) attention_combine_kernel(const AttnArgs a, int n_split, int64_t n_rh) {
    pdl_wait();
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int64_t rh = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (rh >= n_rh) return;
    float m = -INFINITY;
    for (int s = 0; s < n_split; ++s) m = fmaxf(m, a.part_ml[(rh * n_split + s) * 2]);
    float l = 0.f;
    float acc[D / 32];
#pragma unroll
    for (int i = 0; i < D / 32; ++i) acc[i] = 0.f;
    for (int s = 0; s < n_split; ++s) {
        const float ms = a.part_ml[(rh * n_split + s) * 2];
        const float w = ms == -INFINITY ? 0.f : exp2f(ms - m);      // a split all of whose keys were dropped
        l += a.part_ml[(rh * n_split + s) * 2 + 1] * w;
        const float* po = a.part_o + (rh * n_split + s) * D;
#pragma unroll
        for (int i = 0; i < D / 32; ++i) acc[i] += po[i * 32 + lane] * w;
    }
    const float inv = 1.f / l;
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(a.o) + rh * D;   // [B, n, H, d] is contiguous in (row, head)
#pragma unroll
    for (int i = 0; i < D / 32; ++i) out[i * 32 + lane] = __float2bfloat16_rn(acc[i] * inv);
}

// Key splits: enough CTAs to cover the machine about twice when there are few query tiles.
static int attention_splits(int q_ctas, int key_tiles, int* tiles_per_split) {
    int want = q_ctas >= kAttnTargetCtas ? 1 : (kAttnTargetCtas + q_ctas - 1) / q_ctas;
    if (want > key_tiles) want = key_tiles;
    if (want < 1) want = 1;
    *tiles_per_split = (key_tiles + want - 1) / want;
    return (key_tiles + *tiles_per_split - 1) / *tiles_per_split;
}

size_t attention_scratch_bytes(int head_dim) {
    // splits are only used below kAttnTargetCtas query CTAs, and n_split * q_ctas < 2 * kAttnTargetCtas
    return (size_t)2 * kAttnTargetCtas * 64 * (head_dim + 2) * sizeof(float);
}

int launch_attention(const AttnArgs& a, cudaStream_t stream) {
    if (a.batch == 0 || a.n == 0) return 0;
    static const bool no_tc = [] { const char* e = getenv("ACACHE_ATTN_TC"); return e && e[0] == '0'; }();
    if (!no_tc) {
        const int r = launch_attention_tc(a, a.status, stream);
        if (r != 0) return r;
    }
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)a.head_dim);
    const int q_tiles = (a.n + 63) / 64;
    int tps;
    const int n_split = attention_splits(q_tiles * a.n_heads * a.batch, (a.ctx_len + 63) / 64, &tps);
    dim3 grid(q_tiles * n_split, a.n_heads, a.batch);
    const int64_t n_rh = (int64_t)a.batch * a.n * a.n_heads;
    if (a.head_dim == 128) {
        constexpr int SMEM = (1 + 2 * ATT_STAGES) * 64 * 128 * 2;
        cudaFuncSetAttribute(attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        launch_pdl(attention_kernel<128>, grid, 128, SMEM, stream, a, scale_log2e, n_split, tps);
        if (n_split > 1) launch_pdl(attention_combine_kernel<128>, (unsigned)((n_rh + 3) / 4), 128, 0, stream, a, n_split, n_rh);
    } else {
        constexpr int SMEM = (1 + 2 * ATT_STAGES) * 64 * 64 * 2;
        cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        launch_pdl(attention_kernel<64>, grid, 128, SMEM, stream, a, scale_log2e, n_split, tps);
        if (n_split > 1) launch_pdl(attention_combine_kernel<64>, (unsigned)((n_rh + 3) / 4), 128, 0, stream, a, n_split, n_rh);
    }
    return n_split > 1 ? 2 : 1;
}

}  // namespace acache
