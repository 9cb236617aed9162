// Anchor scoring (Eq. 4-5) for head dimension 128 on the 5th-generation tensor cores.  Both passes stream
// the cached affix keys through shared memory by TMA and are bound by that read:
//
//   pass 1, row statistics   S = Q_mask K^T  (M = 128 masked rows of one head, N = 256 keys per stage);
//                            thread = masked row: running maximum and denominator over the normaliser's
//                            key range, one entry per CTA (key split);
//   pass 2, column sums      D = K Q_mask^T  (M = 128 keys, N = the masked rows rounded up to 32);
//                            thread = key: sum over the masked rows of exp2(logit - max_q) / den_q,
//                            a sum over the accumulator's columns, so no thread exchanges anything.
//
// The orientation is swapped between the passes so that each reduction runs along the TMEM columns a
// thread holds.  Rows of the query tile past the last masked row and keys past the range read as zero
// through the tensor maps and are masked out.  No float atomics: results are bitwise reproducible.
// Every mbarrier wait is bounded (status flag kFlagWaitExpired on expiry).
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"
#include "tc_ptx.cuh"

namespace acache {

namespace {

constexpr int ST_THREADS = 192;                 // pass 2: warp 0 TMA, warp 1 MMA, warps 2-5 one thread per key
constexpr int ST_THREADS1 = 320;                // pass 1: eight statistics warps, two per row quarter (64 of a stage's 128 keys each)
constexpr int ST_PANEL128 = 128 * 64 * 2;       // 16 KB: 128 rows x 64 columns
constexpr int ST_Q_BYTES = 2 * ST_PANEL128;     // pass 1: the query tile, 128 rows x 128
constexpr int ST_K_BYTES = 2 * ST_PANEL128;     // 128 keys x 128 per stage (both passes)
// Both kernels are sized so that two CTAs share an SM (about 100 KB of shared memory and 256 TMEM columns
// each): a CTA streams only a few stages, and the second CTA's stream hides the first one's start-up.
constexpr int ST_SMEM1 = ST_Q_BYTES + 2 * ST_K_BYTES + 1024 + 256;
constexpr int CS_STAGES = 2;
constexpr int CS_TABLES = 2048;                 // max and 1 / denominator of up to 256 masked rows
constexpr int kKeysPerCta1 = 1024;              // pass 1: keys per CTA = one statistics entry
constexpr int kTilesPerCta2 = 4;                // pass 2: 128-key tiles per CTA

__device__ __forceinline__ void tma3(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(pol)
        : "memory");
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct ScoreTcArgs {
    float* row_stats;        // [B, H, n_split, m, 2]
    float* head_partial;     // [B, H, L]
    int m, n_heads, n_kv_heads;
    int norm_lo, norm_len, affix_start, affix_len;
    int n_split, cache_shared;
    float scale_log2e;
    uint32_t* status;
};

// ---- pass 1 -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(ST_THREADS1, 2)
score_stats_tc_kernel(const ScoreTcArgs a, const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sQ = base, sK0 = base + ST_Q_BYTES;
    const uint32_t bars = base + ST_Q_BYTES + 2 * ST_K_BYTES;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + ST_Q_BYTES + 2 * ST_K_BYTES + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + ST_Q_BYTES + 2 * ST_K_BYTES + 200);
    // barriers: 0 q_full | 1,2 k_full | 3,4 k_empty | 5,6 s_full | 7,8 s_empty
    auto bar = [&](int i) { return bars + 8 * i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.x, split = blockIdx.y;
    const int mtiles = (a.m + 127) / 128;
    const int b = blockIdx.z / mtiles, mt = blockIdx.z - b * mtiles;
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int kb = a.cache_shared ? 0 : b;
    const int key0 = split * kKeysPerCta1;
    const int n_keys = min(kKeysPerCta1, a.norm_len - key0);
    const int n_stage = (n_keys + 127) / 128;

    if (threadIdx.x == 0) {
        for (int i = 0; i <= 6; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(7), 8); mbar_init(bar(8), 8);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();
    pdl_launch_dependents();

    if (warp == 0 && lane == 0) {
        const uint64_t pol_q = policy_evict_last(), pol_k = policy_evict_last();   // the second pass reads the keys again
        mbar_expect_tx(bar(0), ST_Q_BYTES);
        tma3(sQ, &mapQ, h * 128, mt * 128, b, bar(0), pol_q);
        tma3(sQ + ST_PANEL128, &mapQ, h * 128 + 64, mt * 128, b, bar(0), pol_q);
        bool ok = true;
        for (int st = 0; st < n_stage && ok; ++st) {
            const int s = st & 1;
            if (!(ok = mbar_wait(bar(3 + s), ((st >> 1) & 1) ^ 1, abort_flag))) break;
            mbar_expect_tx(bar(1 + s), ST_K_BYTES);
            const uint32_t dst = sK0 + s * ST_K_BYTES;
            const int row = a.norm_lo + key0 + st * 128;
            tma3(dst, &mapK, kvh * 128, row, kb, bar(1 + s), pol_k);
            tma3(dst + ST_PANEL128, &mapK, kvh * 128 + 64, row, kb, bar(1 + s), pol_k);
        }
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = idesc_bf16(128);
        bool ok = mbar_wait(bar(0), 0, abort_flag);
        for (int st = 0; st < n_stage && ok; ++st) {
            const int s = st & 1;
            const uint32_t par = (st >> 1) & 1;
            if (!(ok = mbar_wait(bar(1 + s), par, abort_flag))) break;
            if (!(ok = mbar_wait(bar(7 + s), par ^ 1, abort_flag))) break;
            tc_fence_after();
            const uint32_t k = sK0 + s * ST_K_BYTES;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint64_t da = smem_desc_sw128(sQ + (ks >> 2) * ST_PANEL128) + (uint64_t)((ks & 3) * 2);
                const uint64_t db = smem_desc_sw128(k + (ks >> 2) * ST_PANEL128) + (uint64_t)((ks & 3) * 2);
                tc_mma(tmem_base + s * 128, da, db, idesc, ks > 0 ? 1u : 0u);
            }
            tc_commit(bar(5 + s));     // s_full
            tc_commit(bar(3 + s));     // k_empty
        }
    } else if (warp >= 2) {
        // thread = (masked row, half of the stage's keys): with few masked rows only the warps of the first
        // row quarter(s) have work, so each row's 128 keys per stage are split over two warps
        const int q = warp & 3, cw = (warp - 2) >> 2;
        const int row = q * 32 + lane;
        const int grow = mt * 128 + row;
        const bool live = (mt * 128 + q * 32) < a.m;        // whole warps past the last masked row only keep the barriers moving
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        float mx = -INFINITY, den = 0.f;
        bool ok = true;
        for (int st = 0; st < n_stage && ok; ++st) {
            const int s = st & 1;
            if (!(ok = mbar_wait(bar(5 + s), (st >> 1) & 1, abort_flag))) break;
            tc_fence_after();
            if (live) {
                const int valid = n_keys - st * 128 - cw * 64;     // keys of this thread's half that exist
                for (int c = 0; c < 2 && c * 32 < valid; ++c) {
                    float v[32];
                    tc_ld32(tmem_base + s * 128 + lane_off + cw * 64 + c * 32, v);
                    const int nv = valid - c * 32;
                    float tm = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        v[i] = i < nv ? v[i] * a.scale_log2e : -INFINITY;
                        tm = fmaxf(tm, v[i]);
                    }
                    const float nm = fmaxf(mx, tm);
                    float part = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) part += ex2(v[i] - nm);
                    den = den * ex2(mx - nm) + part;
                    mx = nm;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(7 + s));   // s_empty
        }
        // merge the two key halves of every row in a fixed order (the K stages are idle by now)
        float2* ex = reinterpret_cast<float2*>(base_ptr + ST_Q_BYTES);
        ex[cw * 128 + row] = make_float2(mx, den);
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (ok && !*abort_flag && cw == 0 && live && grow < a.m) {
            float M = -INFINITY, Dn = 0.f;
            for (int c = 0; c < 2; ++c) M = fmaxf(M, ex[c * 128 + row].x);
            for (int c = 0; c < 2; ++c) Dn += ex[c * 128 + row].y * ex2(ex[c * 128 + row].x - M);
            float* stp = a.row_stats + ((((int64_t)b * a.n_heads + h) * a.n_split + split) * a.m + grow) * 2;
            stp[0] = M;
            stp[1] = Dn;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) {
            atomicOr(a.status, kFlagWaitExpired);
            for (int i = 0; i < 4096; ++i) __nanosleep(64);
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem_base) : "memory");
    }
}

// ---- pass 2 -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(ST_THREADS, 2)
score_colsum_tc_kernel(const ScoreTcArgs a, const int n_pad, const __grid_constant__ CUtensorMap mapQ,
                       const __grid_constant__ CUtensorMap mapK) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    // the query tile: two 64-column panels of q_rows (128 or 256) rows each
    const int q_rows = n_pad <= 128 ? 128 : 256;
    const uint32_t q_panel = (uint32_t)q_rows * 128u, q_bytes = 2u * q_panel;
    const uint32_t tmem_cols = n_pad <= 128 ? 256u : 512u;        // two accumulators of n_pad columns
    const uint32_t sQ = base, sK0 = base + q_bytes;
    float* s_max = reinterpret_cast<float*>(base_ptr + q_bytes + CS_STAGES * ST_K_BYTES);     // [256]
    float* s_inv = s_max + 256;
    const uint32_t bars = base + q_bytes + CS_STAGES * ST_K_BYTES + CS_TABLES;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + q_bytes + CS_STAGES * ST_K_BYTES + CS_TABLES + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + q_bytes + CS_STAGES * ST_K_BYTES + CS_TABLES + 200);
    // barriers: 0 q_full | 1,2 k_full | 4,5 k_empty | 7,8 d_full | 9,10 d_empty
    auto bar = [&](int i) { return bars + 8 * i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.x, chunk = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int kb = a.cache_shared ? 0 : b;
    const int key_tiles = (a.affix_len + 127) / 128;
    const int t0 = chunk * kTilesPerCta2;
    const int n_tiles = min(kTilesPerCta2, key_tiles - t0);

    if (threadIdx.x == 0) {
        for (int i = 0; i <= 8; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(9), 4); mbar_init(bar(10), 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();
    pdl_launch_dependents();

    // combine the split statistics of every masked row (fixed order)
    if (threadIdx.x >= 64) {
        const float* st = a.row_stats + ((int64_t)b * a.n_heads + h) * a.n_split * a.m * 2;
        for (int r = threadIdx.x - 64; r < 256; r += 128) {
            float M = -INFINITY, Dn = 0.f;
            if (r < a.m) {
                for (int s = 0; s < a.n_split; ++s) M = fmaxf(M, st[((int64_t)s * a.m + r) * 2]);
                for (int s = 0; s < a.n_split; ++s)
                    Dn += st[((int64_t)s * a.m + r) * 2 + 1] * ex2(st[((int64_t)s * a.m + r) * 2] - M);
            }
            s_max[r] = r < a.m ? M : 0.f;           // padding rows: logit 0, weight 0
            s_inv[r] = r < a.m ? 1.f / Dn : 0.f;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
    }

    if (warp == 0 && lane == 0) {
        // the last read of the keys by this head; with grouped-query attention the other query heads of the KV head still want them
        const uint64_t pol = a.n_heads == a.n_kv_heads ? policy_evict_first() : policy_evict_last();
        const uint64_t pol_q = policy_evict_last();
        mbar_expect_tx(bar(0), q_bytes);               // whole boxes of 128 rows, zero fill included
        for (int p = 0; p < 2; ++p)
            for (int r = 0; r * 128 < q_rows; ++r)
                tma3(sQ + p * q_panel + r * ST_PANEL128, &mapQ, h * 128 + p * 64, r * 128, b, bar(0), pol_q);
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int s = t % CS_STAGES;
            if (!(ok = mbar_wait(bar(4 + s), ((t / CS_STAGES) & 1) ^ 1, abort_flag))) break;
            mbar_expect_tx(bar(1 + s), ST_K_BYTES);
            const uint32_t dst = sK0 + s * ST_K_BYTES;
            const int row = a.affix_start + (t0 + t) * 128;
            tma3(dst, &mapK, kvh * 128, row, kb, bar(1 + s), pol);
            tma3(dst + ST_PANEL128, &mapK, kvh * 128 + 64, row, kb, bar(1 + s), pol);
        }
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = idesc_bf16(n_pad);
        bool ok = mbar_wait(bar(0), 0, abort_flag);
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int s = t % CS_STAGES, d = t & 1;
            if (!(ok = mbar_wait(bar(1 + s), (t / CS_STAGES) & 1, abort_flag))) break;
            if (!(ok = mbar_wait(bar(9 + d), ((t >> 1) & 1) ^ 1, abort_flag))) break;
            tc_fence_after();
            const uint32_t k = sK0 + s * ST_K_BYTES;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint64_t da = smem_desc_sw128(k + (ks >> 2) * ST_PANEL128) + (uint64_t)((ks & 3) * 2);
                const uint64_t db = smem_desc_sw128(sQ + (ks >> 2) * q_panel) + (uint64_t)((ks & 3) * 2);
                tc_mma(tmem_base + d * (tmem_cols >> 1), da, db, idesc, ks > 0 ? 1u : 0u);
            }
            tc_commit(bar(7 + d));     // d_full
            tc_commit(bar(4 + s));     // k_empty
        }
    } else if (warp >= 2) {
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int d = t & 1;
            if (!(ok = mbar_wait(bar(7 + d), (t >> 1) & 1, abort_flag))) break;
            tc_fence_after();
            float sum = 0.f;
            for (int c = 0; c * 32 < n_pad; ++c) {
                float v[32];
                tc_ld32(tmem_base + d * (tmem_cols >> 1) + lane_off + c * 32, v);
#pragma unroll
                for (int i = 0; i < 32; ++i) sum += ex2(fmaf(v[i], a.scale_log2e, -s_max[c * 32 + i])) * s_inv[c * 32 + i];
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(9 + d));   // d_empty
            const int j = (t0 + t) * 128 + row;
            if (j < a.affix_len) a.head_partial[((int64_t)b * a.n_heads + h) * a.affix_len + j] = sum;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) {
            atomicOr(a.status, kFlagWaitExpired);
            for (int i = 0; i < 4096; ++i) __nanosleep(64);
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ---- one pass: the logits stay in tensor memory ------------------------------------------------------
// With at most 64 masked rows the logits of a whole key range fit in tensor memory in the orientation D = K Q^T
// (thread = key, one column per masked row: 32 or 64 columns per 128-key tile, up to 512 columns), so the cached keys
// are read from HBM ONCE: a cluster of eight CTAs covers the normaliser's key range of one (head, request); every CTA
// streams its eighth through a TMA ring, leaves D of all its tiles in tensor memory and keeps a running column
// maximum per thread; then (i) the CTA's maximum per masked row (a transposing reduction through shared memory),
// (ii) e = exp2(s - that maximum) written back over D, its column sums = the CTA's share of the denominator,
// (iii) the eight CTAs' (maximum, share) meet through distributed shared memory and give each masked row one weight
// w_r = exp2(m_cta - M) / denominator, (iv) every thread adds e_r w_r over its key's columns: the key's column sum.
// One exponential per logit, every sum in a fixed order (bitwise reproducible), no float atomics.
constexpr int S1_CLUSTER = 8;
constexpr int S1_THREADS = 192;                 // warp 0 TMA, warp 1 MMA, warps 2-5 one thread per key
constexpr int S1_MAX_TILES = 16;
// query tile (NP rows x 128: 8 or 16 KB) | key ring, 3 or 2 stages (after the last tile: the transposition buffer [128][65]
// fp32) | tables | barriers.  About 105 KB / 85 KB: two CTAs per SM, which is also what tensor memory allows at up to 256
// columns per CTA; a CTA that needs all 512 columns asks for S1_SMEM_WIDE so that no second CTA can be resident beside it
// (a CTA waiting for tensor memory inside a cluster whose peers wait for it at a cluster barrier would never get it).
template <int NP> struct S1 {
    static constexpr int Q_BYTES = 2 * NP * 128;
    static constexpr int STAGES = NP == 32 ? 3 : 2;
    static constexpr int TAB_OFF = Q_BYTES + STAGES * ST_K_BYTES;
    static constexpr int BAR_OFF = TAB_OFF + 2048;
    static constexpr int SMEM = BAR_OFF + 512 + 1024;
    static_assert(128 * 65 * 4 <= STAGES * ST_K_BYTES, "the transposition buffer reuses the key ring");
};
constexpr int S1_SMEM_WIDE = 120 * 1024;

__device__ __forceinline__ void tc_st32f(uint32_t taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]),
          "f"(v[9]), "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "f"(v[16]), "f"(v[17]),
          "f"(v[18]), "f"(v[19]), "f"(v[20]), "f"(v[21]), "f"(v[22]), "f"(v[23]), "f"(v[24]), "f"(v[25]), "f"(v[26]),
          "f"(v[27]), "f"(v[28]), "f"(v[29]), "f"(v[30]), "f"(v[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_sync_s1() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t local_addr, uint32_t rank) {
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(ra) : "memory");
    return v;
}

// NP: columns per key tile (the masked rows rounded up to 32 or 64); tpc: 128-key tiles per CTA
// csize: CTAs per cluster (1, 2, 4 or 8; the launch sets the cluster dimension to the same number)
template <int NP>
__global__ void __launch_bounds__(S1_THREADS, 2)
score_onepass_tc_kernel(const ScoreTcArgs a, const int tpc, const uint32_t tmem_cols, const int csize,
                        const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    constexpr int S1_STAGES = S1<NP>::STAGES, S1_BAR_OFF = S1<NP>::BAR_OFF;
    const uint32_t sQ = base, sK0 = base + S1<NP>::Q_BYTES;
    float* s_t = reinterpret_cast<float*>(base_ptr + S1<NP>::Q_BYTES);          // [128 keys][65]: per-thread column values
    float* s_w = reinterpret_cast<float*>(base_ptr + S1<NP>::TAB_OFF);          // [64] per-row scalar handed to the key threads
    float* s_part = s_w + 64;                                                   // [4 warps][64] partial column reductions
    float2* s_x = reinterpret_cast<float2*>(s_part + 256);                      // [64] (maximum, denominator share) for the peers
    const uint32_t bars = base + S1_BAR_OFF;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + S1_BAR_OFF + 448);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + S1_BAR_OFF + 456);
    // barriers: 0 q_full | 1..3 k_full | 4..6 k_empty | 8..23 d_full of tile t  (S1_STAGES <= 3)
    auto bar = [&](int i) { return bars + 8 * i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = blockIdx.x % csize, h = blockIdx.x / csize, b = blockIdx.y;
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int kb = a.cache_shared ? 0 : b;
    const int key0 = rank * tpc * 128;                                           // first key of this CTA inside the range
    const int n_keys = max(0, min(tpc * 128, a.norm_len - key0));
    const int n_tiles = (n_keys + 127) / 128;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 8 + S1_MAX_TILES; ++i) mbar_init(bar(i), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();
    pdl_launch_dependents();

    if (warp == 0 && lane == 0) {
        // the keys are read once per query head: with grouped-query attention the other heads of the KV head still want them
        const uint64_t pol = a.n_heads == a.n_kv_heads ? policy_evict_first() : policy_evict_last(), pol_q = policy_evict_last();
        mbar_expect_tx(bar(0), 2 * NP * 128);                                    // two 64-column panels of NP rows
        tma3(sQ, &mapQ, h * 128, 0, b, bar(0), pol_q);
        tma3(sQ + NP * 128, &mapQ, h * 128 + 64, 0, b, bar(0), pol_q);
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int s = t % S1_STAGES;
            if (!(ok = mbar_wait(bar(4 + s), ((t / S1_STAGES) & 1) ^ 1, abort_flag))) break;
            mbar_expect_tx(bar(1 + s), ST_K_BYTES);
            const uint32_t dst = sK0 + s * ST_K_BYTES;
            const int row = a.norm_lo + key0 + t * 128;
            tma3(dst, &mapK, kvh * 128, row, kb, bar(1 + s), pol);
            tma3(dst + ST_PANEL128, &mapK, kvh * 128 + 64, row, kb, bar(1 + s), pol);
        }
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = idesc_bf16(NP);
        bool ok = mbar_wait(bar(0), 0, abort_flag);
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int s = t % S1_STAGES;
            if (!(ok = mbar_wait(bar(1 + s), (t / S1_STAGES) & 1, abort_flag))) break;
            tc_fence_after();
            const uint32_t k = sK0 + s * ST_K_BYTES;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint64_t da = smem_desc_sw128(k + (ks >> 2) * ST_PANEL128) + (uint64_t)((ks & 3) * 2);
                const uint64_t db = smem_desc_sw128(sQ + (ks >> 2) * (NP * 128)) + (uint64_t)((ks & 3) * 2);
                tc_mma(tmem_base + t * NP, da, db, idesc, ks > 0 ? 1u : 0u);
            }
            tc_commit(bar(8 + t));     // d_full of tile t
            tc_commit(bar(4 + s));     // k_empty
        }
    }
    // ---------------- key threads: warps 2-5, thread = key lane; everyone meets at the barriers ----------------
    const bool keyw = warp >= 2;
    const int q = warp & 3, kl = q * 32 + lane;                                  // this thread's TMEM lane = key inside a tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    bool ok = true;
    // (i) running maximum per column over this thread's keys, as the tiles arrive
    float cmax[NP];
#pragma unroll
    for (int r = 0; r < NP; ++r) cmax[r] = -INFINITY;
    if (keyw) {
        for (int t = 0; t < n_tiles && ok; ++t) {
            if (!(ok = __all_sync(0xffffffffu, mbar_wait(bar(8 + t), 0, abort_flag)))) break;
            tc_fence_after();
            // the tensor-memory load is collective (.sync.aligned): every lane executes the same one, a lane whose key lies
            // past the range only leaves the values out of its maximum
            const bool there = t * 128 + kl < n_keys;
#pragma unroll
            for (int c = 0; c < NP / 32; ++c) {
                float v[32];
                tc_ld32(tmem_base + lane_off + t * NP + c * 32, v);
#pragma unroll
                for (int i = 0; i < 32; ++i) cmax[c * 32 + i] = there ? fmaxf(cmax[c * 32 + i], v[i]) : cmax[c * 32 + i];
            }
        }
#pragma unroll
        for (int r = 0; r < NP; ++r) s_t[kl * 65 + r] = cmax[r];
    }
    __syncthreads();
    // transposing reduction: key thread kl takes column kl % NP over 128 * NP / 128 keys, then NP threads combine the parts
    constexpr int GROUPS = 128 / NP, KPG = NP;                                   // key groups, keys per group
    if (keyw) {
        const int r = kl % NP, g = kl / NP;
        float m = -INFINITY;
#pragma unroll 8
        for (int k = 0; k < KPG; ++k) m = fmaxf(m, s_t[(g * KPG + k) * 65 + r]);
        s_part[g * 64 + r] = m;
    }
    __syncthreads();
    if (threadIdx.x < NP) {
        float m = -INFINITY;
#pragma unroll
        for (int g = 0; g < GROUPS; ++g) m = fmaxf(m, s_part[g * 64 + threadIdx.x]);
        s_w[threadIdx.x] = m * a.scale_log2e;                                    // the CTA's maximum of row r, in log2 units
    }
    __syncthreads();
    // (ii) e = exp2(s - maximum), written back over D; per-thread column sums
    if (keyw) {
        float csum[NP];
#pragma unroll
        for (int r = 0; r < NP; ++r) csum[r] = 0.f;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const bool there = t * 128 + kl < n_keys;
#pragma unroll
            for (int c = 0; c < NP / 32; ++c) {
                float v[32];
                tc_ld32(tmem_base + lane_off + t * NP + c * 32, v);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float mr = s_w[c * 32 + i];
                    v[i] = (there && mr > -INFINITY) ? ex2(fmaf(v[i], a.scale_log2e, -mr)) : 0.f;
                    csum[c * 32 + i] += v[i];
                }
                tc_st32f(tmem_base + lane_off + t * NP + c * 32, v);
            }
        }
#pragma unroll
        for (int r = 0; r < NP; ++r) s_t[kl * 65 + r] = csum[r];
    }
    __syncthreads();
    if (keyw) {
        const int r = kl % NP, g = kl / NP;
        float d = 0.f;
#pragma unroll 8
        for (int k = 0; k < KPG; ++k) d += s_t[(g * KPG + k) * 65 + r];
        s_part[g * 64 + r] = d;
    }
    __syncthreads();
    if (threadIdx.x < NP) {
        float d = 0.f;
#pragma unroll
        for (int g = 0; g < GROUPS; ++g) d += s_part[g * 64 + threadIdx.x];
        s_x[threadIdx.x] = make_float2(s_w[threadIdx.x], d);
    }
    // (iii) the eight CTAs' statistics meet: one weight per masked row
    cluster_sync_s1();
    if (threadIdx.x < NP) {
        float2 st[S1_CLUSTER];
#pragma unroll
        for (int c = 0; c < S1_CLUSTER; ++c)
            st[c] = c < csize ? ld_cluster_f2(smem_u32(s_x + threadIdx.x), (uint32_t)c) : make_float2(-INFINITY, 0.f);
        float M = -INFINITY, Dn = 0.f;
#pragma unroll
        for (int c = 0; c < S1_CLUSTER; ++c) M = fmaxf(M, st[c].x);
#pragma unroll
        for (int c = 0; c < S1_CLUSTER; ++c)
            if (st[c].x > -INFINITY) Dn += st[c].y * ex2(st[c].x - M);
        const float mine = s_x[threadIdx.x].x;
        s_part[threadIdx.x] = ((int)threadIdx.x < a.m && mine > -INFINITY && Dn > 0.f) ? ex2(mine - M) / Dn : 0.f;
    }
    __syncthreads();
    // (iv) the key's column sum
    if (keyw) {
        for (int t = 0; t < n_tiles && ok; ++t) {
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < NP / 32; ++c) {
                float v[32];
                tc_ld32(tmem_base + lane_off + t * NP + c * 32, v);
#pragma unroll
                for (int i = 0; i < 32; ++i) sum = fmaf(v[i], s_part[c * 32 + i], sum);
            }
            const int j = a.norm_lo + key0 + t * 128 + kl - a.affix_start;     // position inside the affix
            if (t * 128 + kl < n_keys && j >= 0 && j < a.affix_len)
                a.head_partial[((int64_t)b * a.n_heads + h) * a.affix_len + j] = sum;
        }
    }
    tc_fence_before();
    cluster_sync_s1();            // no CTA leaves while a peer may still read its statistics
    if (*abort_flag) {
        if (threadIdx.x == 0) {
            atomicOr(a.status, kFlagWaitExpired);
            for (int i = 0; i < 4096; ++i) __nanosleep(64);
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

}  // namespace

int score_tc_splits(int norm_len) { return (norm_len + kKeysPerCta1 - 1) / kKeysPerCta1; }

// Launches the two passes; 0 if the problem is not for these kernels (the caller uses the mma.sync ones).
int launch_score_tc(const ScoreArgs& a, uint32_t* status, cudaStream_t stream) {
    if (a.head_dim != 128 || a.m > 256 || a.m <= 0 || !status) return 0;
    if ((a.kv_batch_stride * 2) % 16) return 0;
    static const bool off = [] { const char* e = getenv("ACACHE_SCORE_TC"); return e && e[0] == '0'; }();
    if (off) return 0;
    // measured (m = 32): the mma.sync kernels win while there is little to read (L = 512, B = 1: 16 against 20 us),
    // these from about two thousand keys up (L = 2048: 23 against 28 us; L = 8192: 38 against 74 us)
    static const int min_keys = [] { const char* e = getenv("ACACHE_SCORE_TC_MIN_KEYS"); return e ? atoi(e) : 2048; }();
    if ((int64_t)a.batch * a.norm_len < min_keys) return 0;
    const bool shared = a.kv_batch_stride == 0;
    const int kv_cols = a.n_kv_heads * 128;
    const int ctx_rows = a.norm_lo + a.norm_len > a.affix_start + a.affix_len ? a.norm_lo + a.norm_len : a.affix_start + a.affix_len;
    std::lock_guard<std::mutex> lock(g_map3_mutex);
    CUtensorMap map_q, map_k;
    const CUtensorMap* mq = get_map3(a.q_mask, a.m, a.n_heads * 128, a.batch, (int64_t)a.m * a.n_heads * 128);
    if (!mq) return 0;
    map_q = *mq; mq = &map_q;        // the cache may replace the entry at the next lookup
    const CUtensorMap* mk = get_map3(a.cache_k, ctx_rows, kv_cols, shared ? 1 : a.batch,
                                     shared ? (int64_t)ctx_rows * kv_cols : a.kv_batch_stride);
    if (!mk) return 0;
    map_k = *mk; mk = &map_k;
    static bool attr = false;
    if (!attr) {
        cudaFuncSetAttribute(score_stats_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ST_SMEM1);
        cudaFuncSetAttribute(score_colsum_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             2 * 256 * 128 + CS_STAGES * ST_K_BYTES + CS_TABLES + 1024 + 256);
        attr = true;
    }
    static const bool onepass_on = [] { const char* e = getenv("ACACHE_SCORE_ONEPASS"); return !e || atoi(e) != 0; }();
    if (onepass_on && a.m <= 64) {
        // One pass, logits kept in tensor memory.  A (head, request) pair's key range is cut over a cluster of csize CTAs:
        // as few as tensor memory allows (256 columns per CTA keep two CTAs on an SM) once the pairs alone fill the
        // machine, more when there are few pairs (measured: at L = 512, B = 8 eight CTAs of half a tile each took 51 us
        // where the two-pass kernels take 24).
        const int np = a.m <= 32 ? 32 : 64;
        const int tiles = (a.norm_len + 127) / 128;
        int csize = 1;
        while (csize < S1_CLUSTER && ((tiles + csize - 1) / csize) * np > 256) csize <<= 1;        // tensor memory
        while (csize < S1_CLUSTER && csize * 2 <= tiles && (int64_t)a.n_heads * a.batch * csize < 2 * 148) csize <<= 1;   // fill
        // ACACHE_SCORE_CLUSTER = 1, 2, 4 or 8 forces the cluster size wherever tensor memory allows it (the tests run
        // every size over the same cases, ragged and empty key ranges included)
        static const int forced = [] { const char* e = getenv("ACACHE_SCORE_CLUSTER"); return e ? atoi(e) : 0; }();
        if ((forced == 1 || forced == 2 || forced == 4 || forced == 8) && ((tiles + forced - 1) / forced) * np <= 512) csize = forced;
        const int tpc = (tiles + csize - 1) / csize;
        if (tpc * np <= 512 && (tpc >= 2 || forced)) {
            uint32_t cols = 32;
            while ((int)cols < tpc * np) cols <<= 1;
            const CUtensorMap* mq1 = get_map3(a.q_mask, a.m, a.n_heads * 128, a.batch, (int64_t)a.m * a.n_heads * 128, np);
            if (mq1) {
                const CUtensorMap map_q1 = *mq1;
                static bool attr1 = false;
                if (!attr1) {
                    cudaFuncSetAttribute(score_onepass_tc_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, S1_SMEM_WIDE);
                    cudaFuncSetAttribute(score_onepass_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, S1_SMEM_WIDE);
                    attr1 = true;
                }
                ScoreTcArgs t1{};
                t1.row_stats = a.row_stats; t1.head_partial = a.head_partial;
                t1.m = a.m; t1.n_heads = a.n_heads; t1.n_kv_heads = a.n_kv_heads;
                t1.norm_lo = a.norm_lo; t1.norm_len = a.norm_len; t1.affix_start = a.affix_start; t1.affix_len = a.affix_len;
                t1.n_split = 1; t1.cache_shared = shared ? 1 : 0;
                t1.scale_log2e = 1.4426950408889634f / sqrtf(128.f);
                t1.status = status;
                cudaLaunchConfig_t cfg{};
                cfg.gridDim = dim3(a.n_heads * csize, a.batch);
                cfg.blockDim = dim3(S1_THREADS);
                cfg.dynamicSmemBytes = cols > 256 ? (size_t)S1_SMEM_WIDE : (size_t)(np == 32 ? S1<32>::SMEM : S1<64>::SMEM);
                cfg.stream = stream;
                cudaLaunchAttribute at[2];
                at[0].id = cudaLaunchAttributeClusterDimension;
                at[0].val.clusterDim.x = csize; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
                at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
                at[1].val.programmaticStreamSerializationAllowed = 1;
                cfg.attrs = at;
                cfg.numAttrs = 2;
                const cudaError_t e1 = np == 32
                    ? cudaLaunchKernelEx(&cfg, score_onepass_tc_kernel<32>, t1, tpc, cols, csize, map_q1, *mk)
                    : cudaLaunchKernelEx(&cfg, score_onepass_tc_kernel<64>, t1, tpc, cols, csize, map_q1, *mk);
                return e1 == cudaSuccess ? 1 : -1;
            }
        }
    }
    ScoreTcArgs t{};
    t.row_stats = a.row_stats; t.head_partial = a.head_partial;
    t.m = a.m; t.n_heads = a.n_heads; t.n_kv_heads = a.n_kv_heads;
    t.norm_lo = a.norm_lo; t.norm_len = a.norm_len; t.affix_start = a.affix_start; t.affix_len = a.affix_len;
    t.n_split = score_tc_splits(a.norm_len); t.cache_shared = shared ? 1 : 0;
    t.scale_log2e = 1.4426950408889634f / sqrtf(128.f);
    t.status = status;
    const int mtiles = (a.m + 127) / 128;
    if (launch_pdl(score_stats_tc_kernel, dim3(a.n_heads, t.n_split, a.batch * mtiles), dim3(ST_THREADS1), ST_SMEM1, stream, t, *mq,
                   *mk) != cudaSuccess)
        return -1;
    const int n_pad = (a.m + 31) & ~31;
    const int key_tiles = (a.affix_len + 127) / 128;
    const int cs_smem = 2 * (n_pad <= 128 ? 128 : 256) * 128 + CS_STAGES * ST_K_BYTES + CS_TABLES + 1024 + 256;
    if (launch_pdl(score_colsum_tc_kernel, dim3(a.n_heads, (key_tiles + kTilesPerCta2 - 1) / kTilesPerCta2, a.batch),
                   dim3(ST_THREADS), cs_smem, stream, t, n_pad, *mq, *mk) != cudaSuccess)
        return -1;
    return 2;
}

}  // namespace acache
