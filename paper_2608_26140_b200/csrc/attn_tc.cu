// Bidirectional attention of many recomputed rows over the whole context (Section 4.3) on the
// 5th-generation tensor cores.  Two kernels share the scheme below: attention_tc_kernel (one CTA = 128
// query rows of one head; used when a request has at most 128 rows) and attention_tc2q_kernel (one CTA
// = 256 query rows, described where it is defined).  Key/value tiles of 128 keys stream through shared
// memory by TMA (3-d tensor maps: positions past the context end and rows past the request's row count
// read as zero).
//
//   S = Q K^T    tcgen05.mma 128 x 128 x 16, both operands K-major, into a TMEM buffer
//   softmax      scaled max, exp2, running denominator; P is written as packed bf16 over the low
//                columns of its S buffer, so it never passes through shared memory
//   O += P V     tcgen05.mma 128 x 128 x 16, A = P read from tensor memory, B = V read in place as an
//                MN-major operand (token-major V rows are contiguous along the head dimension)
//
// One-tile kernel: sixteen softmax warps, four threads per query row (32 keys each), two S buffers: the
// S of tile j+1 is issued before the softmax of tile j is consumed, so tensor work overlaps the
// exponentials.  The running maximum used for the exponent is only raised (and O rescaled in
// TMEM) when the true maximum has grown by more than 2^8, which keeps P within bf16 range and
// makes rescales rare.  Every mbarrier wait is bounded (status flag kFlagWaitExpired on expiry).
// With two key sources (a cache shared by the batch + each request's private rows, Section 4.1) the
// private rows' tiles follow the cache's, and key masks tell which of the two serves a position; when
// every request brings at most 32 rows (decode passes), four requests share one tile, one per 32-row
// quarter, so that the shared cache's tiles are read once per four requests.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"
#include "tc_ptx.cuh"

namespace acache {

constexpr int AT_THREADS = 608;                  // warp 0: TMA, warp 1: S MMAs, warps 2-17: softmax (four threads per row), warp 18: PV MMAs
constexpr int AT_TILE = 128 * 128 * 2;           // 32 KB: a [128 x 128] bf16 tile as two 64-column panels
constexpr int AT_PANEL = 128 * 64 * 2;           // 16 KB
constexpr int AT_SLACK = 256;                    // the dynamic window starts 1024-aligned in practice; checked at run time
constexpr int AT_SMEM = 5 * AT_TILE + AT_SLACK + 256;   // Q, K x2, V x2 (P lives in tensor memory)
constexpr float kRescaleGap = 8.f;               // log2 units

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* map, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]),
          "f"(v[9]), "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "f"(v[16]), "f"(v[17]),
          "f"(v[18]), "f"(v[19]), "f"(v[20]), "f"(v[21]), "f"(v[22]), "f"(v[23]), "f"(v[24]), "f"(v[25]), "f"(v[26]),
          "f"(v[27]), "f"(v[28]), "f"(v[29]), "f"(v[30]), "f"(v[31])
        : "memory");
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^x on the FMA pipe for x <= ~8 (Cody-Waite: x = n + f with n = rint(x), |f| <= 0.5; a cubic for 2^f
// with relative error 7.5e-5, far below the bf16 rounding of P; n goes straight into the exponent).
// A quarter of the exponentials take this route so that the MUFU pipe is not the only one working.
__device__ __forceinline__ float poly_exp2(float x) {
    x = fmaxf(x, -126.f);
    const float t = x + 12582912.f;                 // 1.5 * 2^23: the low mantissa bits now hold rint(x)
    const float f = x - (t - 12582912.f);
    const float p = fmaf(fmaf(fmaf(0.05517146f, f, 0.24261086f), f, 0.69326097f), f, 0.9999281f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}
// D += A B with A read from tensor memory (rows = TMEM lanes, two bf16 of consecutive K per 32-bit column)
__device__ __forceinline__ void tc_mma_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// MN-major bf16 operand with the 128-byte swizzle: rows of the K index are 128 bytes (64 elements
// of the MN index), 8-row groups 1024 bytes apart (stride byte offset), and the next 64 elements
// of the MN index start one 16 KB panel further (leading byte offset).
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t saddr) {
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(AT_PANEL >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

struct AttnTcArgs {
    void* o;                  // bf16 [B, n, H*d]
    int n, ctx_len, n_heads, n_kv_heads;
    float scale_log2e;
    uint32_t* status;
    // two key sources (shared storage + private rows, Section 4.1): after the cache's tiles come the tiles of
    // the fresh rows [B, n, Hkv, d]; pos_excl masks the cache positions those rows serve, row_keep the fresh
    // rows that do not serve their position (duplicates).  n_fresh_tiles = 0: the cache alone; pos_excl may then
    // still name cache positions that do not exist as keys (the DropNA layout of Section 5.3).
    int n_fresh_tiles, excl_words, keep_words, cache_shared;
    int kv_prefetch;          // two-query-tile kernel: K/V tiles requested into L2 ahead of the rings
    // one-tile kernel over a shared cache with at most 32 rows per request (decode passes): group = 4 puts the rows
    // of four requests into the four 32-row quarters of one tile, so that the shared cache's key tiles are read
    // once per four requests; each request's fresh tiles follow, visible to its own quarter only.  Else 1.
    int group, batch;
    const uint32_t* pos_excl;
    const uint32_t* row_keep;
    // Eq. 4-5 taken from this attention's own logits (two-query-tile kernel; the one-shot probe of Section 3.2): for the
    // query rows flagged in score_rowmask [B, rm_words] (bit i = compact row i is a masked position) the kernel keeps,
    // next to the softmax denominator, the same sum restricted to the affix keys, and after the last key tile walks the
    // affix key tiles once more with the product turned round (D = K Q^T: thread = key, columns = query rows), adding
    // exp2(s - reference) / denominator over the flagged rows.  score_partial [B, H, q_tiles, L]: per (head, 128-row
    // query tile) column sums, written only by tiles that hold flagged rows.
    const uint32_t* score_rowmask;
    float* score_partial;
    int rm_words, q_tiles, affix_start, affix_len;
    int score_norm_full;      // weight = 1 / the full denominator (Eq. 4 over every key) instead of the affix keys' share
};

// Wait for the two-query-tile kernel's threads whose hand-overs sit on the critical path of every key tile (the thread that
// issues the tensor-core instructions, the softmax threads waiting for S): no sleep between polls (the many-row attention
// went from 785 to 748 us on a 14 752-row layer; the one-tile kernel did not change); bounded like every wait.
__device__ __forceinline__ bool mbar_spin(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < (TC_WAIT_LIMIT << 4); ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 4095u) == 4095u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__global__ void __launch_bounds__(AT_THREADS, 1)
attention_tc_kernel(const AttnTcArgs a, const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                    const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapKn,
                    const __grid_constant__ CUtensorMap mapVn) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ uint16_t row_max[2][4][128];  // [tile parity][key quarter][row]: upper halves of fp32, rounded up
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    if (base - smem_u32(smem_raw) > (uint32_t)AT_SLACK) {      // the tiles would not fit: report, touch nothing
        if (threadIdx.x == 0) atomicOr(a.status, kFlagWaitExpired);
        return;
    }
    const uint32_t sQ = base, sK0 = base + AT_TILE, sV0 = base + 3 * AT_TILE;
    const uint32_t bars = base + 5 * AT_TILE;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + 5 * AT_TILE + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + 5 * AT_TILE + 200);
    // barriers: 0 q_full | 1,2 k_full | 3,4 k_empty | 5,6 v_full | 7,8 v_empty | 9,10 s_full | 11,12 unused |
    //           13,14 p_full | 15,16 pv_done (P V of the tile completed: O holds it, its S/P buffer is free)
    auto bar = [&](int i) { return bars + 8 * i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int n_cache_tiles = (a.ctx_len + 127) / 128;
    const int n_tiles = n_cache_tiles + a.n_fresh_tiles * min(a.group, a.batch - (int)blockIdx.z * a.group);
    const int kb = a.cache_shared ? 0 : b;          // one cache for the whole batch, or one per request
    const int G = a.group;                          // requests per tile (4: blockIdx.z counts groups of four)
    const int b0 = b * G;                           // first request of the tile
    const int n_req = min(G, a.batch - b0);
    // 32-row quarters of the tile that hold rows: the softmax warps of the others have nothing to do (their
    // rows of S, P and O are never read), which matters when a decode pass brings 32 rows per request
    const int live_q = G > 1 ? n_req : min(4, (a.n - qt * 128 + 31) / 32);

    if (threadIdx.x == 0) {
        for (int i = 0; i <= 10; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(13), 4 * live_q); mbar_init(bar(14), 4 * live_q);    // p_full: the softmax warps that have rows
        mbar_init(bar(15), 1); mbar_init(bar(16), 1);      // pv_done
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tS0 = tmem_base, tO = tmem_base + 256;
    pdl_wait();
    pdl_launch_dependents();

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer ----------------
        const uint64_t pol_q = policy_evict_first(), pol_kv = policy_evict_last();
        if (G > 1) {
            // 32-row boxes: request b0 + r fills rows [32 r, 32 r + 32) of both panels (rows past its n read as zero)
            mbar_expect_tx(bar(0), n_req * 8192);
            for (int r = 0; r < n_req; ++r) {
                tma_load_3d(sQ + r * 4096, &mapQ, h * 128, 0, b0 + r, bar(0), pol_q);
                tma_load_3d(sQ + AT_PANEL + r * 4096, &mapQ, h * 128 + 64, 0, b0 + r, bar(0), pol_q);
            }
        } else {
            mbar_expect_tx(bar(0), AT_TILE);
            tma_load_3d(sQ, &mapQ, h * 128, qt * 128, b, bar(0), pol_q);
            tma_load_3d(sQ + AT_PANEL, &mapQ, h * 128 + 64, qt * 128, b, bar(0), pol_q);
        }
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int s = j & 1;
            const uint32_t par = ((j >> 1) & 1) ^ 1;
            if (!(ok = mbar_wait(bar(3 + s), par, abort_flag))) break;
            const bool fresh = j >= n_cache_tiles;
            const CUtensorMap* mk = fresh ? &mapKn : &mapK;
            const CUtensorMap* mv = fresh ? &mapVn : &mapV;
            const int f = j - n_cache_tiles;                          // fresh tiles: request by request
            const int r0 = (fresh ? f % a.n_fresh_tiles : j) * 128, bz = fresh ? b0 + f / a.n_fresh_tiles : kb;
            mbar_expect_tx(bar(1 + s), AT_TILE);
            tma_load_3d(sK0 + s * AT_TILE, mk, kvh * 128, r0, bz, bar(1 + s), pol_kv);
            tma_load_3d(sK0 + s * AT_TILE + AT_PANEL, mk, kvh * 128 + 64, r0, bz, bar(1 + s), pol_kv);
            if (!(ok = mbar_wait(bar(7 + s), par, abort_flag))) break;
            mbar_expect_tx(bar(5 + s), AT_TILE);
            tma_load_3d(sV0 + s * AT_TILE, mv, kvh * 128, r0, bz, bar(5 + s), pol_kv);
            tma_load_3d(sV0 + s * AT_TILE + AT_PANEL, mv, kvh * 128 + 64, r0, bz, bar(5 + s), pol_kv);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer 1: S = Q K^T (M 128, N 128, both operands K-major) ----------------
        // The two products are issued by two threads of different warps: one thread doing both spends
        // more time in its four barrier waits and sixteen issues per tile than the tensor pipe needs
        // for the work.  Every tcgen05.commit tracks the issuing thread's own MMAs, and the cross
        // dependencies (P of tile j after S of tile j, S buffer reuse, O in tile order) all go through
        // mbarriers, so no ordering between the two threads is assumed.
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        bool ok = mbar_wait(bar(0), 0, abort_flag);
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int s = j & 1;
            const uint32_t par = (j >> 1) & 1;
            if (!(ok = mbar_wait(bar(1 + s), par, abort_flag))) break;          // K of tile j landed
            // its S buffer also holds the P of tile j - 2: free once that tile's P V has completed
            if (j >= 2 && !(ok = mbar_wait(bar(15 + s), ((j - 2) >> 1) & 1, abort_flag))) break;
            tc_fence_after();
            const uint32_t k = sK0 + s * AT_TILE;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint64_t da = smem_desc_sw128(sQ + (ks >> 2) * AT_PANEL) + (uint64_t)((ks & 3) * 2);
                const uint64_t db = smem_desc_sw128(k + (ks >> 2) * AT_PANEL) + (uint64_t)((ks & 3) * 2);
                tc_mma(tS0 + s * 128, da, db, idesc_s, ks > 0 ? 1u : 0u);
            }
            tc_commit(bar(9 + s));     // s_full
            tc_commit(bar(3 + s));     // k_empty
        }
    } else if (warp == AT_THREADS / 32 - 1 && lane == 0) {
        // ---------------- MMA issuer 2: O += P V (A = P K-major, B = V MN-major) ----------------
        const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int s = j & 1;
            if (!(ok = mbar_wait(bar(13 + s), (j >> 1) & 1, abort_flag))) break;    // P of tile j written, O rescaled
            if (!(ok = mbar_wait(bar(5 + s), (j >> 1) & 1, abort_flag))) break;     // V of tile j landed
            tc_fence_after();
            const uint32_t v = sV0 + s * AT_TILE;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint64_t db = smem_desc_mn_sw128(v + ks * 2048);
                tc_mma_ta(tO, tS0 + s * 128 + ks * 8, db, idesc_o, (j > 0 || ks > 0) ? 1u : 0u);   // 16 keys = 8 columns of P
            }
            tc_commit(bar(15 + s));    // pv_done: O holds tiles 0..j, the S/P buffer is free
            tc_commit(bar(7 + s));     // v_empty
        }
    } else if (warp >= 2 && warp < 18 && (warp & 3) < live_q) {
        // ---------------- softmax: four threads per query row ----------------
        // Warp 2 + 4 c + q' (q = warp & 3 is its TMEM lane quarter) takes keys [32 c, 32 c + 32) of every
        // tile for the 32 rows of quarter q, and columns [32 c, 32 c + 32) of O.  Sixteen warps (four per
        // scheduler) keep the exponential, conversion and TMEM-load latencies of one warp hidden behind
        // the others.  The four threads of a row agree on the row maximum through shared memory once per
        // tile.  The four warps of a row quarter meet at a named barrier every tile, so they only ever
        // leave the loop together: a wait that ran out sets the abort flag, the thread skips its work,
        // and everyone breaks after the next barrier.
        const int c4 = (warp - 2) >> 2;
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        const uint32_t col_off = (uint32_t)(c4 * 32);
        const int bq = G > 1 ? b0 + q : b;          // the request whose rows this quarter holds
        float m_use = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j & 1;
            // which of this thread's 32 keys count: the cache's positions up to the context end, minus those a
            // fresh row serves; of the fresh rows, those that serve their position
            uint32_t keep;
            if (j < n_cache_tiles) {
                const int valid = a.ctx_len - j * 128 - c4 * 32;
                keep = valid >= 32 ? 0xffffffffu : (valid <= 0 ? 0u : (1u << valid) - 1u);
                if (a.pos_excl && j * 4 + c4 < a.excl_words) keep &= ~__ldg(a.pos_excl + (int64_t)bq * a.excl_words + j * 4 + c4);
            } else {
                const int f = j - n_cache_tiles;
                if (G > 1 && f / a.n_fresh_tiles != q) {
                    // another request's fresh rows: none of them is a key of this quarter's rows.  All four warps
                    // of the quarter come here, so none of them goes to the quarter's barrier for this tile.
                    if (ok && (ok = mbar_wait(bar(9 + s), (j >> 1) & 1, abort_flag))) {
                        tc_fence_after();
                        uint32_t pz[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) pz[i] = 0u;
                        tc_st16(tS0 + s * 128 + c4 * 16 + lane_off, pz);
                        tc_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(13 + s));
                    }
                    continue;
                }
                const int w = (f % a.n_fresh_tiles) * 4 + c4;
                keep = w < a.keep_words ? __ldg(a.row_keep + (int64_t)bq * a.keep_words + w) : 0u;
            }
            float sv[32];
            float mt = -INFINITY;
            if (ok && (ok = mbar_wait(bar(9 + s), (j >> 1) & 1, abort_flag))) {
                tc_fence_after();
                // this thread's quarter row of S into registers, then the S buffer is free for tile j + 2
                tc_ld32(tS0 + s * 128 + col_off + lane_off, sv);
                float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                if (keep == 0xffffffffu) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], sv[i]);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if ((keep >> i) & 1u) m4[i & 3] = fmaxf(m4[i & 3], sv[i]);
                }
                mt = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * a.scale_log2e;
            }
            // the four threads of a row must use the same number: all take the largest of the four
            // quarter-row maxima rounded up to 16 significant bits (an upper bound is all the exponent needs)
            uint32_t mb = __float_as_uint(mt);
            if ((mb & 0xFFFFu) && !(mb >> 31)) mb += 0x10000u;
            mb >>= 16;
            row_max[s][c4][row] = (uint16_t)mb;
            asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");     // the four warps that share these 32 rows
            if (*abort_flag) { ok = false; break; }
            mt = fmaxf(fmaxf(__uint_as_float((uint32_t)row_max[s][0][row] << 16), __uint_as_float((uint32_t)row_max[s][1][row] << 16)),
                       fmaxf(__uint_as_float((uint32_t)row_max[s][2][row] << 16), __uint_as_float((uint32_t)row_max[s][3][row] << 16)));
            bool raise = false;
            if (j == 0) {
                m_use = mt;
            } else if (mt - m_use > kRescaleGap) {
                raise = true;
            }
            if (__any_sync(0xffffffffu, raise)) {
                // O may only be touched once the P V of tile j - 1 has completed
                if ((ok = mbar_wait(bar(15 + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag))) {
                    tc_fence_after();
                    const float f = raise ? fast_exp2(m_use - mt) : 1.f;
                    float v[32];
                    tc_ld32(tO + lane_off + col_off, v);
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] *= f;
                    tc_st32(tO + lane_off + col_off, v);
                    tc_wait_st();
                    l *= f;
                    if (raise) m_use = mt;
                }
            }
            if (!ok) continue;
            // P overwrites the S buffer in tensor memory: 32 keys = 16 columns of two bf16 at column 16 c4
            // (every thread of the row has read its S columns: they all passed the barrier above)
            float l4[4] = {0.f, 0.f, 0.f, 0.f};
            if (keep == 0xffffffffu) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float x = fmaf(sv[i], a.scale_log2e, -m_use);
                    const float p = (i & 3) == 3 ? poly_exp2(x) : fast_exp2(x);
                    l4[i & 3] += p;
                    sv[i] = p;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float p = ((keep >> i) & 1u) ? fast_exp2(fmaf(sv[i], a.scale_log2e, -m_use)) : 0.f;
                    l4[i & 3] += p;
                    sv[i] = p;
                }
            }
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(sv[2 * i], sv[2 * i + 1]);
            tc_st16(tS0 + s * 128 + c4 * 16 + lane_off, pk);
            tc_wait_st();
            l += (l4[0] + l4[1]) + (l4[2] + l4[3]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(13 + s));   // p_full
        }
        // epilogue: O / l once the last P V has completed; the denominators of the four quarters add up
        if (ok && n_tiles > 0) ok = mbar_wait(bar(15 + ((n_tiles - 1) & 1)), ((n_tiles - 1) >> 1) & 1, abort_flag);
        float* row_sum = reinterpret_cast<float*>(base_ptr + AT_TILE);         // the K stages are idle now
        row_sum[c4 * 128 + row] = l;
        asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");
        if (ok && !*abort_flag) {
            tc_fence_after();
            const int grow = G > 1 ? lane : qt * 128 + row;     // the row inside its request
            const float inv = 1.f / ((row_sum[row] + row_sum[128 + row]) + (row_sum[256 + row] + row_sum[384 + row]));
            __nv_bfloat16* out = static_cast<__nv_bfloat16*>(a.o) + (((int64_t)bq * a.n + grow) * a.n_heads + h) * 128 + col_off;
            float v[32];
            tc_ld32(tO + lane_off + col_off, v);
            if (grow < a.n) {
#pragma unroll
                for (int k8 = 0; k8 < 4; ++k8) {
                    const float* pv = v + k8 * 8;
                    *reinterpret_cast<uint4*>(out + k8 * 8) =
                        make_uint4(pack_bf16(pv[0] * inv, pv[1] * inv), pack_bf16(pv[2] * inv, pv[3] * inv),
                                   pack_bf16(pv[4] * inv, pv[5] * inv), pack_bf16(pv[6] * inv, pv[7] * inv));
                }
            }
        }
    }
    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) {
            atomicOr(a.status, kFlagWaitExpired);
            for (int i = 0; i < 4096; ++i) __nanosleep(64);   // let copies already in flight land
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

// ---- two query tiles per CTA ------------------------------------------------------------------
// 256 query rows of one head share every K/V tile that lands in shared memory.  Each 128-row query tile
// has its own S buffer, O accumulator and softmax warps (one thread per row: the row maximum needs no
// exchange).  The softmax works through a tile's 128 keys in two halves of 64 (so that a row's values
// fit in registers without spilling) and writes each half's P over the low columns of the S buffer; one
// thread issues everything: the P V of a half as soon as that half's P is there, and after the second
// half the tile's next S into the same buffer (the tensor pipe executes one thread's instructions in
// order).  While one query tile's softmax runs, the tensor pipe works on the other's.  Measured and not
// kept: S as two 64-key products into two buffers per query tile (a 128 x 64 x 16 product holds the
// issuing thread as long as a 128 x 128 x 16 one: 74 against 66 cycles), and one issuing thread per query
// tile (their interleaved instructions ran slower than one thread's fixed order).
//
// The exponent reference of a row only moves when a half's maximum exceeds it by more than 2^8 (then O
// and the denominator are rescaled), so the common path is: x = s * scale - reference (two per FFMA2),
// maximum, exp2 (a quarter of them on the FMA pipe), bf16 pack, store to tensor memory.
constexpr int AT2_THREADS = 320;                 // warp 0: TMA, warp 1: MMA issuer, warps 2-5 / 6-9: softmax of query tile 0 / 1
constexpr int AT2_SMEM = 6 * AT_TILE + AT_SLACK + 256 + 2048;   // Q x2, K x2, V x2, barriers, score tables

__device__ __forceinline__ void tc_ld32_nowait(uint32_t taddr, float (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]),
          "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15]), "=f"(v[16]),
          "=f"(v[17]), "=f"(v[18]), "=f"(v[19]), "=f"(v[20]), "=f"(v[21]), "=f"(v[22]), "=f"(v[23]), "=f"(v[24]),
          "=f"(v[25]), "=f"(v[26]), "=f"(v[27]), "=f"(v[28]), "=f"(v[29]), "=f"(v[30]), "=f"(v[31])
        : "r"(taddr)
        : "memory");
}
// The loads above are complete after this; the values pass through it so that no use can move ahead of it.
__device__ __forceinline__ void tc_wait_ld32(float (&v)[32]) {
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7]), "+f"(v[8]),
          "+f"(v[9]), "+f"(v[10]), "+f"(v[11]), "+f"(v[12]), "+f"(v[13]), "+f"(v[14]), "+f"(v[15]), "+f"(v[16]),
          "+f"(v[17]), "+f"(v[18]), "+f"(v[19]), "+f"(v[20]), "+f"(v[21]), "+f"(v[22]), "+f"(v[23]), "+f"(v[24]),
          "+f"(v[25]), "+f"(v[26]), "+f"(v[27]), "+f"(v[28]), "+f"(v[29]), "+f"(v[30]), "+f"(v[31])
        :
        : "memory");
}
__device__ __forceinline__ void tc_st32u(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
          "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
          "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}

__global__ void __launch_bounds__(AT2_THREADS, 1)
attention_tc2q_kernel(const AttnTcArgs a, const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                      const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapKn,
                      const __grid_constant__ CUtensorMap mapVn) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    if (base - smem_u32(smem_raw) > (uint32_t)AT_SLACK) {      // the tiles would not fit: report, touch nothing
        if (threadIdx.x == 0) atomicOr(a.status, kFlagWaitExpired);
        return;
    }
    const uint32_t sQ = base, sK0 = base + 2 * AT_TILE, sV0 = base + 4 * AT_TILE;
    const uint32_t bars = base + 6 * AT_TILE;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + 6 * AT_TILE + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + 6 * AT_TILE + 200);
    // barriers: 0 q_full | 1,2 k_full | 3,4 k_empty | 5,6 v_full | 7,8 v_empty | 9 + t: s_full |
    //           11 + 2 t + hb: p_full | 15 + 2 t + hb: pv_done   (query tile t, key half hb)
    auto bar = [&](int i) { return bars + 8 * i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (a.n_heads / a.n_kv_heads);
    const int n_cache_tiles = (a.ctx_len + 127) / 128;
    const int n_tiles = n_cache_tiles + a.n_fresh_tiles;
    const int kb = a.cache_shared ? 0 : b;
    const int n_sets = (qt * 256 + 128 < a.n) ? 2 : 1;      // the last CTA of an odd tile count has one tile
    float2* s_tab = reinterpret_cast<float2*>(base_ptr + 6 * AT_TILE + 256);     // [2 query tiles][128 rows] (reference, weight)

    if (threadIdx.x == 0) {
        for (int i = 0; i <= 10; ++i) mbar_init(bar(i), 1);
        for (int i = 11; i <= 14; ++i)                         // p_full: the softmax warps of the query tile that have rows
            mbar_init(bar(i), max(1, min(4, (a.n - qt * 256 - (i >= 13 ? 128 : 0) + 31) / 32)));
        for (int i = 15; i <= 18; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(19), 4); mbar_init(bar(20), 4);          // score sweep: the four warps of a query tile are done with D
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // columns: S of query tile 0 | S of query tile 1 | O of query tile 0 | O of query tile 1, 128 each
    pdl_wait();
    pdl_launch_dependents();
    // score sweep (Eq. 4-5 from this attention's logits): only CTAs whose 256 query rows hold a flagged row walk the
    // affix key tiles [sw0, sw0 + n_sw) a second time
    int n_sw = 0, sw0 = 0;
    if (a.score_rowmask && a.affix_len > 0) {
        uint32_t any = 0u;
        for (int w = qt * 8; w < min(qt * 8 + 8, a.rm_words); ++w) any |= __ldg(a.score_rowmask + (int64_t)b * a.rm_words + w);
        if (any) { sw0 = a.affix_start >> 7; n_sw = ((a.affix_start + a.affix_len - 1) >> 7) - sw0 + 1; }
    }

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer ----------------
        const uint64_t pol_q = policy_evict_first(), pol_kv = policy_evict_last();
        mbar_expect_tx(bar(0), n_sets * AT_TILE);
        for (int t = 0; t < n_sets; ++t) {
            tma_load_3d(sQ + t * AT_TILE, &mapQ, h * 128, qt * 256 + t * 128, b, bar(0), pol_q);
            tma_load_3d(sQ + t * AT_TILE + AT_PANEL, &mapQ, h * 128 + 64, qt * 256 + t * 128, b, bar(0), pol_q);
        }
        // K/V tiles a few iterations ahead are requested into L2, so that the loads into the two-stage rings
        // (issued one iteration before use) do not wait on HBM
        auto prefetch_tile = [&](int j) {
            if (j >= n_tiles) return;
            const bool fresh = j >= n_cache_tiles;
            const int r0 = (fresh ? j - n_cache_tiles : j) * 128, bz = fresh ? b : kb;
            tma_prefetch_3d(fresh ? &mapKn : &mapK, kvh * 128, r0, bz);
            tma_prefetch_3d(fresh ? &mapKn : &mapK, kvh * 128 + 64, r0, bz);
            tma_prefetch_3d(fresh ? &mapVn : &mapV, kvh * 128, r0, bz);
            tma_prefetch_3d(fresh ? &mapVn : &mapV, kvh * 128 + 64, r0, bz);
        };
        for (int j = 2; j < 2 + a.kv_prefetch; ++j) prefetch_tile(j);
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int s = j & 1;
            const uint32_t par = ((j >> 1) & 1) ^ 1;
            if (a.kv_prefetch) prefetch_tile(j + 2 + a.kv_prefetch);
            if (!(ok = mbar_wait(bar(3 + s), par, abort_flag))) break;
            const bool fresh = j >= n_cache_tiles;
            const CUtensorMap* mk = fresh ? &mapKn : &mapK;
            const CUtensorMap* mv = fresh ? &mapVn : &mapV;
            const int r0 = (fresh ? j - n_cache_tiles : j) * 128, bz = fresh ? b : kb;
            mbar_expect_tx(bar(1 + s), AT_TILE);
            tma_load_3d(sK0 + s * AT_TILE, mk, kvh * 128, r0, bz, bar(1 + s), pol_kv);
            tma_load_3d(sK0 + s * AT_TILE + AT_PANEL, mk, kvh * 128 + 64, r0, bz, bar(1 + s), pol_kv);
            if (!(ok = mbar_wait(bar(7 + s), par, abort_flag))) break;
            mbar_expect_tx(bar(5 + s), AT_TILE);
            tma_load_3d(sV0 + s * AT_TILE, mv, kvh * 128, r0, bz, bar(5 + s), pol_kv);
            tma_load_3d(sV0 + s * AT_TILE + AT_PANEL, mv, kvh * 128 + 64, r0, bz, bar(5 + s), pol_kv);
        }
        for (int js = 0; js < n_sw && ok; ++js) {            // the affix key tiles once more (keys only)
            const int jj = n_tiles + js, s = jj & 1;
            if (!(ok = mbar_wait(bar(3 + s), ((jj >> 1) & 1) ^ 1, abort_flag))) break;
            mbar_expect_tx(bar(1 + s), AT_TILE);
            tma_load_3d(sK0 + s * AT_TILE, &mapK, kvh * 128, (sw0 + js) * 128, kb, bar(1 + s), pol_kv);
            tma_load_3d(sK0 + s * AT_TILE + AT_PANEL, &mapK, kvh * 128 + 64, (sw0 + js) * 128, kb, bar(1 + s), pol_kv);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer ----------------
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint32_t idesc_o = idesc_s | (1u << 16);       // B = V is MN-major
        auto issue_s = [&](int t, int j) {                   // S_t = Q_t K_j^T, then s_full of query tile t
            const uint32_t k = sK0 + (j & 1) * AT_TILE;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint64_t da = smem_desc_sw128(sQ + t * AT_TILE + (ks >> 2) * AT_PANEL) + (uint64_t)((ks & 3) * 2);
                const uint64_t db = smem_desc_sw128(k + (ks >> 2) * AT_PANEL) + (uint64_t)((ks & 3) * 2);
                tc_mma(tmem_base + t * 128, da, db, idesc_s, ks > 0 ? 1u : 0u);
            }
            tc_commit(bar(9 + t));
        };
        bool ok = mbar_spin(bar(0), 0, abort_flag);
        if (ok && n_tiles > 0 && (ok = mbar_spin(bar(1), 0, abort_flag))) {
            tc_fence_after();
            for (int t = 0; t < n_sets; ++t) issue_s(t, 0);
            tc_commit(bar(3));                               // k_empty of stage 0
        }
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int s = j & 1;
            const bool more = j + 1 < n_tiles;
            if (!(ok = mbar_spin(bar(5 + s), (j >> 1) & 1, abort_flag))) break;                       // V of tile j landed
            if (more && !(ok = mbar_spin(bar(1 + (s ^ 1)), ((j + 1) >> 1) & 1, abort_flag))) break;   // K of tile j + 1 landed
            const uint32_t v = sV0 + s * AT_TILE;
            for (int t = 0; t < n_sets && ok; ++t) {
                for (int hb = 0; hb < 2 && ok; ++hb) {
                    if (!(ok = mbar_spin(bar(11 + 2 * t + hb), j & 1, abort_flag))) break;  // P of this half written, O rescaled
                    tc_fence_after();
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) {
                        const int ks = hb * 4 + k4;          // 16 keys = 8 columns of P
                        tc_mma_ta(tmem_base + 256 + t * 128, tmem_base + t * 128 + ks * 8, smem_desc_mn_sw128(v + ks * 2048), idesc_o,
                                  (j > 0 || ks > 0) ? 1u : 0u);
                    }
                    tc_commit(bar(15 + 2 * t + hb));         // pv_done: O holds everything up to this half
                }
                if (ok && more) issue_s(t, j + 1);           // overwrites P: executes after the P V just issued
            }
            tc_commit(bar(7 + s));                           // v_empty
            if (more) tc_commit(bar(3 + (s ^ 1)));           // k_empty of tile j + 1
        }
        // score sweep: D_t = K Q_t^T into the S buffer of query tile t (its last P V was issued above by this thread, and
        // the tensor pipe keeps one thread's instructions in order)
        for (int js = 0; js < n_sw && ok; ++js) {
            const int jj = n_tiles + js, s = jj & 1;
            if (!(ok = mbar_spin(bar(1 + s), (jj >> 1) & 1, abort_flag))) break;
            const uint32_t k = sK0 + s * AT_TILE;
            for (int t = 0; t < n_sets && ok; ++t) {
                if (js > 0 && !(ok = mbar_spin(bar(19 + t), (js - 1) & 1, abort_flag))) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t da = smem_desc_sw128(k + (ks >> 2) * AT_PANEL) + (uint64_t)((ks & 3) * 2);
                    const uint64_t db = smem_desc_sw128(sQ + t * AT_TILE + (ks >> 2) * AT_PANEL) + (uint64_t)((ks & 3) * 2);
                    tc_mma(tmem_base + t * 128, da, db, idesc_s, ks > 0 ? 1u : 0u);
                }
                tc_commit(bar(9 + t));
            }
            if (ok) tc_commit(bar(3 + s));                   // k_empty
        }
    } else if (warp >= 2 && warp < 2 + 4 * n_sets) {
      const int t = (warp - 2) >> 2;
      const int q = warp & 3;                              // the warp's TMEM lane quarter
      const int row = q * 32 + lane;
      const uint32_t lane_off = (uint32_t)(q * 32) << 16;
      const uint32_t tS = tmem_base + t * 128 + lane_off, tO = tmem_base + 256 + t * 128 + lane_off;
      const bool has_rows = q * 32 < a.n - qt * 256 - t * 128;
      // Eq. 4 normalises over the affix keys: the denominator restricted to them is kept next to the full one
      const bool want_lf = n_sw > 0 && !a.score_norm_full;
      float m_use = -INFINITY, l = 0.f, lf = 0.f;
      bool ok = true;
      if (has_rows) {
        // ---------------- softmax: one thread per query row ----------------
        const float2 sc2 = make_float2(a.scale_log2e, a.scale_log2e);
        for (int i = 0; i < 2 * n_tiles && ok; ++i) {
            const int hb = i & 1, j = i >> 1;
            // which of the half's 64 keys count: the cache's positions up to the context end, minus those a
            // fresh row serves; of the fresh rows, those that serve their position
            uint32_t keep[2];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int w = hb * 2 + c;
                if (j < n_cache_tiles) {
                    const int valid = a.ctx_len - j * 128 - w * 32;
                    keep[c] = valid >= 32 ? 0xffffffffu : (valid <= 0 ? 0u : (1u << valid) - 1u);
                    if (a.pos_excl && j * 4 + w < a.excl_words) keep[c] &= ~__ldg(a.pos_excl + (int64_t)b * a.excl_words + j * 4 + w);
                } else {
                    const int fw = (j - n_cache_tiles) * 4 + w;
                    keep[c] = fw < a.keep_words ? __ldg(a.row_keep + (int64_t)b * a.keep_words + fw) : 0u;
                }
            }
            // of those keys, the ones inside the affix span (cache tiles only): all, none, or some (then the slow path)
            uint32_t aff[2] = {0u, 0u};
            if (want_lf && j < n_cache_tiles) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int k0 = j * 128 + (hb * 2 + c) * 32;
                    const int lo = max(a.affix_start - k0, 0), hi = min(a.affix_start + a.affix_len - k0, 32);
                    if (hi > lo) aff[c] = (hi - lo >= 32 ? 0xffffffffu : ((1u << (hi - lo)) - 1u) << lo);
                }
            }
            const bool aff_all = (aff[0] & aff[1]) == 0xffffffffu, aff_none = (aff[0] | aff[1]) == 0u;
            const bool all = (keep[0] & keep[1]) == 0xffffffffu && (aff_all || aff_none);
            // warp-uniform: the tensor-memory accesses below are collective
            if (hb == 0) {
                if (!(ok = __all_sync(0xffffffffu, mbar_spin(bar(9 + t), j & 1, abort_flag)))) break;
                tc_fence_after();
            }
            float sv[2][32];
            tc_ld32_nowait(tS + hb * 64, sv[0]);
            tc_ld32_nowait(tS + hb * 64 + 32, sv[1]);
            tc_wait_ld32(sv[0]);
            tc_wait_ld32(sv[1]);
            // x = s * scale - reference, in place; the reference is 0 until a half with a key that counts
            const bool first = m_use == -INFINITY;
            const float m_ref = first ? 0.f : m_use;
            const float2 mr2 = make_float2(-m_ref, -m_ref);
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float2 r = __ffma2_rn(make_float2(sv[c][2 * e], sv[c][2 * e + 1]), sc2, mr2);
                    sv[c][2 * e] = r.x;
                    sv[c][2 * e + 1] = r.y;
                }
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            if (all) {
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e) m4[e & 3] = fmaxf(m4[e & 3], sv[c][e]);
            } else {
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if ((keep[c] >> e) & 1u) m4[e & 3] = fmaxf(m4[e & 3], sv[c][e]);
            }
            const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
            const bool raise = mx > kRescaleGap || (first && mx > -INFINITY);
            if (__any_sync(0xffffffffu, raise)) {
                const float f = raise ? (first ? 0.f : fast_exp2(-mx)) : 1.f;
                if (i > 0) {
                    // O may only be touched once the P V of half i - 1 (and with it every earlier one) has completed
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait(bar(15 + 2 * t + ((i - 1) & 1)), ((i - 1) >> 1) & 1, abort_flag)))) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        float v[32];
                        tc_ld32(tO + c * 32, v);
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] *= f;
                        tc_st32(tO + c * 32, v);
                    }
                    tc_wait_st();
                }
                l *= f;
                lf *= f;
                if (raise) {
                    m_use = m_ref + mx;
#pragma unroll
                    for (int c = 0; c < 2; ++c)
#pragma unroll
                        for (int e = 0; e < 32; ++e) sv[c][e] -= mx;
                }
            }
            // P as packed bf16: the half's 64 keys go to columns 32 hb .. 32 hb + 31 of the S buffer, over S values of
            // keys below 64 that this thread read in the first half
            float2 l2a = make_float2(0.f, 0.f), l2b = make_float2(0.f, 0.f), lf2 = make_float2(0.f, 0.f);
            uint32_t pk[32];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                if (all) {
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        const float2 pa = make_float2(fast_exp2(sv[c][e]), fast_exp2(sv[c][e + 1]));
                        const float2 pb = make_float2(fast_exp2(sv[c][e + 2]), poly_exp2(sv[c][e + 3]));
                        l2a = __fadd2_rn(l2a, pa);
                        l2b = __fadd2_rn(l2b, pb);
                        pk[c * 16 + (e >> 1)] = pack_bf16(pa.x, pa.y);
                        pk[c * 16 + (e >> 1) + 1] = pack_bf16(pb.x, pb.y);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const float p0 = ((keep[c] >> e) & 1u) ? fast_exp2(sv[c][e]) : 0.f;
                        const float p1 = ((keep[c] >> (e + 1)) & 1u) ? fast_exp2(sv[c][e + 1]) : 0.f;
                        l2a = __fadd2_rn(l2a, make_float2(p0, p1));
                        lf2 = __fadd2_rn(lf2, make_float2(((aff[c] >> e) & 1u) ? p0 : 0.f, ((aff[c] >> (e + 1)) & 1u) ? p1 : 0.f));
                        pk[c * 16 + (e >> 1)] = pack_bf16(p0, p1);
                    }
                }
            }
            tc_st32u(tS + hb * 32, pk);
            tc_wait_st();
            const float half_sum = (l2a.x + l2a.y) + (l2b.x + l2b.y);
            l += half_sum;
            lf += all ? (aff_all ? half_sum : 0.f) : (lf2.x + lf2.y);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(11 + 2 * t + hb));   // p_full
        }
        // epilogue: O / l once the last P V has completed
        if (ok && n_tiles > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(15 + 2 * t + 1), (n_tiles - 1) & 1, abort_flag));
        if (ok) {
            tc_fence_after();
            const int grow = qt * 256 + t * 128 + row;
            const float inv = 1.f / l;
            __nv_bfloat16* out = static_cast<__nv_bfloat16*>(a.o) + (((int64_t)b * a.n + grow) * a.n_heads + h) * 128;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                float v[32];
                tc_ld32(tO + c * 32, v);
                if (grow < a.n) {
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8) {
                        const float* pv = v + k8 * 8;
                        *reinterpret_cast<uint4*>(out + c * 32 + k8 * 8) =
                            make_uint4(pack_bf16(pv[0] * inv, pv[1] * inv), pack_bf16(pv[2] * inv, pv[3] * inv),
                                       pack_bf16(pv[4] * inv, pv[5] * inv), pack_bf16(pv[6] * inv, pv[7] * inv));
                    }
                }
            }
        }
      }
      if (n_sw > 0) {
        // ---------------- score sweep: thread = key, columns = the query rows of tile t ----------------
        // every row's (reference, weight): weight = 1 / (its denominator over the affix keys) for a flagged row, else 0
        {
            const int grow = qt * 256 + t * 128 + row;
            float w = 0.f;
            const float den = a.score_norm_full ? l : lf;
            if (has_rows && ok && grow < a.n && den > 0.f &&
                ((__ldg(a.score_rowmask + (int64_t)b * a.rm_words + (grow >> 5)) >> (grow & 31)) & 1u))
                w = 1.f / den;
            s_tab[t * 128 + row] = make_float2(has_rows && m_use > -INFINITY ? m_use : 0.f, w);
        }
        asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");     // the four warps of query tile t
        uint32_t nz = 0u;                                              // 32-row column chunks that hold a flagged row
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (__any_sync(0xffffffffu, s_tab[t * 128 + c * 32 + lane].y != 0.f)) nz |= 1u << c;
        for (int js = 0; js < n_sw; ++js) {
            if (!__all_sync(0xffffffffu, mbar_wait(bar(9 + t), (n_tiles + js) & 1, abort_flag))) break;
            tc_fence_after();
            float sum = 0.f;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                if (!((nz >> c) & 1u)) continue;
                float v[32];
                tc_ld32(tS + c * 32, v);
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float2 mw = s_tab[t * 128 + c * 32 + e];
                    sum += fast_exp2(fmaf(v[e], a.scale_log2e, -mw.x)) * mw.y;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(19 + t));
            const int key = (sw0 + js) * 128 + row, jrel = key - a.affix_start;
            if (jrel >= 0 && jrel < a.affix_len)
                a.score_partial[(((int64_t)b * a.n_heads + h) * a.q_tiles + qt * 2 + t) * a.affix_len + jrel] = sum;
        }
      }
    }
    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) {
            atomicOr(a.status, kFlagWaitExpired);
            for (int i = 0; i < 4096; ++i) __nanosleep(64);   // let copies already in flight land
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

// ---- host side ------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn3() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

// bf16 [batch, rows, cols] with row stride = cols and the given batch stride (elements);
// box = 64 cols x 128 rows x 1, 128-byte swizzle, zero fill out of bounds.
struct Map3Key { const void* ptr; int rows, cols, batch; int64_t bstride; int box_rows; };
struct Map3Entry { Map3Key key; CUtensorMap map; };
constexpr int kMap3Cache = 1024;
std::mutex g_map3_mutex;   // guards the cache below; a returned pointer is only good until the next lookup: callers copy the map
Map3Entry g_maps3[kMap3Cache];
int g_map3_count = 0, g_map3_next = 0;

const CUtensorMap* get_map3(const void* ptr, int rows, int cols, int batch, int64_t bstride, int box_rows) {
    for (int i = 0; i < g_map3_count; ++i) {
        const Map3Key& k = g_maps3[i].key;
        if (k.ptr == ptr && k.rows == rows && k.cols == cols && k.batch == batch && k.bstride == bstride && k.box_rows == box_rows)
            return &g_maps3[i].map;
    }
    EncodeTiledFn fn = encode_fn3();
    if (!fn) return nullptr;
    Map3Entry& e = g_maps3[g_map3_next];
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)batch};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)bstride * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    if (fn(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return nullptr;
    e.key = Map3Key{ptr, rows, cols, batch, bstride, box_rows};
    g_map3_next = (g_map3_next + 1) % kMap3Cache;
    if (g_map3_count < kMap3Cache) ++g_map3_count;
    return &e.map;
}


namespace {
}  // namespace

// Returns the number of kernels launched, 0 if this problem is not for the tensor-core kernel
// (the caller then uses the mma.sync kernel), -1 if a launch failed.
int launch_attention_tc(const AttnArgs& a, uint32_t* status, cudaStream_t stream) {
    if (a.head_dim != 128 || a.batch == 0 || a.n == 0) return 0;
    // reads through the position -> row map become two key sources when the key masks came with it
    const bool two_src = a.slot && a.pos_excl && a.row_keep && a.k_new && a.v_new;
    if (a.slot && !two_src) return 0;
    const int q_tiles = (a.n + 127) / 128;
    // measured at batch 1 with 26-4096 rows over 600-8300 keys: never slower than the key-split mma.sync
    // kernel, even with a single query tile per head (32 CTAs)
    static const int min_ctas = [] { const char* e = getenv("ACACHE_ATTN_TC_MIN_CTAS"); return e ? atoi(e) : 1; }();
    if ((int64_t)q_tiles * a.n_heads * a.batch < min_ctas) return 0;
    if ((a.kv_batch_stride * 2) % 16) return 0;
    const bool shared = a.kv_batch_stride == 0;           // one cache for the whole batch
    const int kv_cols = a.n_kv_heads * 128;
    std::lock_guard<std::mutex> lock(g_map3_mutex);
    // decode passes over a shared cache: the rows of four requests share one tile (see AttnTcArgs::group)
    static const bool group_on = [] { const char* e = getenv("ACACHE_ATTN_GROUP"); return !e || atoi(e) != 0; }();
    const int group = (group_on && two_src && shared && a.n <= 32 && a.batch >= 2) ? 4 : 1;
    CUtensorMap maps[5];
    const CUtensorMap* found[5];
    found[0] = get_map3(a.q, a.n, a.n_heads * 128, a.batch, (int64_t)a.n * a.n_heads * 128, group > 1 ? 32 : 128);
    if (found[0]) maps[0] = *found[0];
    found[1] = get_map3(a.cache_k, a.ctx_len, kv_cols, shared ? 1 : a.batch, shared ? (int64_t)a.ctx_len * kv_cols : a.kv_batch_stride);
    if (found[1]) maps[1] = *found[1];
    found[2] = get_map3(a.cache_v, a.ctx_len, kv_cols, shared ? 1 : a.batch, shared ? (int64_t)a.ctx_len * kv_cols : a.kv_batch_stride);
    if (found[2]) maps[2] = *found[2];
    const int n_fresh = a.n_fresh ? a.n_fresh : a.n;
    found[3] = two_src ? get_map3(a.k_new, n_fresh, kv_cols, a.batch, (int64_t)n_fresh * kv_cols) : found[1];
    if (found[3]) maps[3] = two_src ? *found[3] : maps[1];
    found[4] = two_src ? get_map3(a.v_new, n_fresh, kv_cols, a.batch, (int64_t)n_fresh * kv_cols) : found[2];
    if (found[4]) maps[4] = two_src ? *found[4] : maps[2];
    const CUtensorMap *mq = found[0] ? &maps[0] : nullptr, *mk = found[1] ? &maps[1] : nullptr, *mv = found[2] ? &maps[2] : nullptr,
                      *mkn = found[3] ? &maps[3] : nullptr, *mvn = found[4] ? &maps[4] : nullptr;
    if (!mq || !mk || !mv || !mkn || !mvn) return 0;
    static bool attr = false;
    if (!attr) {
        cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM);
        cudaFuncSetAttribute(attention_tc2q_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT2_SMEM);
        attr = true;
    }
    AttnTcArgs t{};
    t.o = a.o; t.n = a.n; t.ctx_len = a.ctx_len; t.n_heads = a.n_heads; t.n_kv_heads = a.n_kv_heads;
    t.scale_log2e = 1.4426950408889634f / sqrtf(128.f);
    t.status = status;
    t.cache_shared = shared ? 1 : 0;
    t.group = group; t.batch = a.batch;
    if (two_src) {
        t.n_fresh_tiles = (n_fresh + 127) / 128; t.excl_words = a.excl_words; t.keep_words = a.keep_words;
        t.pos_excl = a.pos_excl; t.row_keep = a.row_keep;      // with key_drop the caller has OR-ed it into pos_excl
    } else if (a.key_drop) {
        t.excl_words = a.excl_words; t.pos_excl = a.key_drop;
    }
    t.kv_prefetch = 2;        // K/V tiles requested into L2 this many iterations ahead of the two-stage rings
    // Two query tiles per CTA pay off when the halved grid still fills the SMs and the context is short enough
    // for the per-CTA prologue and epilogue to matter (measured, one against the other: 2048-2560 keys with
    // 1000+ rows, 8-15 % faster; 8192 keys, 5-10 % slower; fewer CTAs than SMs, up to 1.8x slower).
    // ACACHE_ATTN_TC2Q = 0: never, 2: whenever there are two tiles.
    static const int mode_2q = [] { const char* e = getenv("ACACHE_ATTN_TC2Q"); return e ? atoi(e) : 1; }();
    const bool fused_score = a.score_rowmask && a.score_partial && group == 1;
    if (fused_score) {
        t.score_rowmask = a.score_rowmask; t.score_partial = a.score_partial; t.rm_words = a.rm_words; t.q_tiles = q_tiles;
        t.affix_start = a.affix_start; t.affix_len = a.affix_len; t.score_norm_full = a.score_norm_full;
    }
    // the scores are taken from the logits in the two-query-tile kernel only
    const bool use_2q = fused_score || mode_2q == 2 || (mode_2q == 1 && a.ctx_len + (two_src ? n_fresh : 0) <= 4096 &&
                                                        (int64_t)((q_tiles + 1) / 2) * a.n_heads * a.batch >= 148);
    cudaError_t err;
    if (use_2q && (q_tiles >= 2 || fused_score))
        err = launch_pdl(attention_tc2q_kernel, dim3((q_tiles + 1) / 2, a.n_heads, a.batch), dim3(AT2_THREADS), AT2_SMEM, stream, t,
                         *mq, *mk, *mv, *mkn, *mvn);
    else
        err = launch_pdl(attention_tc_kernel, dim3(q_tiles, a.n_heads, (a.batch + group - 1) / group), dim3(AT_THREADS), AT_SMEM,
                         stream, t, *mq, *mk, *mv, *mkn, *mvn);
    return err == cudaSuccess ? 1 : -1;
}

}  // namespace acache
