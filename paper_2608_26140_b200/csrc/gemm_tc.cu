// C[M, N] = A[M, K] * B[N, K]^T (bf16 in, fp32 accumulate) on the 5th-generation tensor
// cores for the projections of the selective recomputation (Section 3.3).
//
// gemm_tc_kernel (at most one CTA per SM):
//   phase 0 (optional)  gather the rows of R (or take compact rows) and RMSNorm them into the
//                       A operand, then a grid-wide barrier
//   phase 1             the contraction: work = (output tiles of 128 x 256) x (K blocks of 64),
//                       the flat list of (tile, k-block) iterations cut into equal contiguous
//                       ranges, one per CTA, so every SM streams the same number of weight
//                       bytes whatever N and K are.  One thread issues TMA loads into a 4-stage
//                       128-byte-swizzled ring (weights evict-first, activations evict-last in
//                       L2), one thread issues tcgen05.mma (128 x 256 x 16) into one of two TMEM
//                       accumulators, four warps drain TMEM with tcgen05.ld and write fp32
//                       partial tiles
// gemm_tc2_kernel (two or more 128-row tiles): a cluster of two CTAs per 256 x 256 tile,
//   tcgen05.mma.cta_group::2; whole tiles walked round-robin, or, when the tiles fill less than
//   two thirds of a wave, equal contiguous (tile, k-block) ranges per cluster like the kernel above.
// gemm_finish_kernel: sums the partial tiles of every output element in ascending CTA order
//   (bitwise reproducible) and applies the epilogue: bias + RoPE + KV scatter, residual add,
//   or SwiGLU.  It is a kernel of its own because it is bound by L2 latency and wants far
//   more threads in flight than one CTA per SM provides (measured: fused into the contraction
//   kernel behind a second grid barrier it was ~10 us slower per projection).
//
// Every wait (mbarrier or grid barrier) is bounded: on expiry the CTA raises kFlagWaitExpired
// in the status word, stops issuing work, lets its in-flight copies land, frees its TMEM and
// returns.  The grid never exceeds the SM count, so all CTAs are resident for the barrier.
#include <cuda.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "kernels.h"
#include "launch.h"
#include "rows.cuh"
#include "tc_ptx.cuh"

namespace acache {

constexpr int TC_BM = 128, TC_BN = 256, TC_BK = 64, TC_STAGES = 4;
constexpr int TC_A_BYTES = TC_BM * TC_BK * 2;          // 16 KB
constexpr int TC_HALF_BYTES = 128 * TC_BK * 2;         // 16 KB: one 128-row half of the B tile
constexpr int TC_STAGE_BYTES = TC_A_BYTES + 2 * TC_HALF_BYTES;
constexpr int TC_THREADS = 192;                        // warp 0: TMA, warp 1: MMA, warps 2-5: drain; all six warps do phase 0
constexpr int TC_SMEM = TC_STAGES * TC_STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int TC_SLOT_FLOATS = TC_BM * TC_BN;          // one fp32 partial tile
constexpr uint32_t GRID_WAIT_LIMIT = 1u << 21;

struct TcPlan {
    int m_tiles, n_tiles, KB, tiles, U, ctas, smax;
    int prefetch;         // K blocks past the ring whose weight tiles are requested into L2 before the dependency wait
    int prefill;          // ring stages whose weight halves are loaded before the dependency wait
    int pair_u;           // two-SM kernel, stream-K mode: (pair tile, K block) iterations per cluster (0: whole tiles)
    int m_pairs;          // 256-row tile rows of the two-SM kernel
    int units;            // 128-row B halves over all segments (non-SwiGLU) or ffn/128 (SwiGLU)
    int group_n;          // two-SM kernel, whole tiles: weight tiles per group of the tile order
    int w_keep;           // weights loaded with the evict-last policy (every row tile re-reads them from L2) instead of evict-first
};

// Which weight matrix and row the 128-row half `h` of N tile `nt` starts at; -1 if past the end.
__device__ __forceinline__ int half_source(const GemmArgs& g, const TcPlan& p, int nt, int h, int& row) {
    if (g.epilogue == kEpiSwiGLU) {
        row = nt * 128;
        return h;                      // half 0: gate rows, half 1: up rows
    }
    int u = nt * 2 + h;
    if (u >= p.units) return -1;
    int r = u * 128, seg = 0;
    while (seg < 2 && r >= g.n[seg]) { r -= g.n[seg]; ++seg; }
    row = r;
    return seg;
}

// Grid-wide barrier number `k` (1, 2, ...) of this launch on a pair of counters in global
// memory: arrivals only ever add to bar[0], so barrier k is passed at k * gridDim.x.  Bounded;
// returns false (and raises the CTA's abort flag) if the others do not arrive.
// self_test: the failure-detection self-test (acache_debug_expire_next_wait): the target is one arrival more than
// the grid can deliver and the poll limit is short, so the wait runs out and the abort path below is taken.
__device__ __forceinline__ bool grid_barrier(unsigned int* bar, unsigned int k, volatile int* abort_flag, bool self_test = false) {
    __syncthreads();
    if (threadIdx.x == 0 && !*abort_flag) {
        __threadfence();
        atomicAdd(&bar[0], 1u);
        const unsigned int target = k * gridDim.x + (self_test ? 1u : 0u);
        const uint32_t limit = self_test ? (1u << 12) : GRID_WAIT_LIMIT;
        bool ok = false;
        for (uint32_t i = 0; i < limit; ++i) {
            unsigned int v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(bar) : "memory");
            if (v >= target) { ok = true; break; }
            __nanosleep(i < 64 ? 20 : 100);
        }
        if (!ok) *abort_flag = 1;
        __threadfence();
    }
    __syncthreads();
    return !*abort_flag;
}

__device__ __forceinline__ uint4 pack8(const float* v) {
    return make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}

// ---- epilogues on W adjacent fp32 accumulator columns of one row (W = 16 or 32) ----------------
// Every store is W*2 bytes of one row: whole 32-byte sectors, no partial-sector writes.

// out[grow, col..col+W) = bf16(resid[grow] + acc)
template <int W>
__device__ __forceinline__ void out_residual(const GemmArgs& g, int grow, int col, float (&v)[W]) {
    const int N = g.n[0];
    const int64_t roff = g.resid_off ? __ldcg(g.resid_off + grow) : (int64_t)grow * N;
    const uint4* rp = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(g.resid) + roff + col);
    uint4* o = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(g.c) + (int64_t)grow * N + col);
#pragma unroll
    for (int j = 0; j < W / 8; ++j) {
        const uint4 r = __ldcg(rp + j);
        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { v[8 * j + 2 * i] += bf16_lo(rw[i]); v[8 * j + 2 * i + 1] += bf16_hi(rw[i]); }
        o[j] = pack8(v + 8 * j);
    }
}

// out[grow, col..col+W) = bf16(silu(gate) * up)
template <int W>
__device__ __forceinline__ void out_swiglu(const GemmArgs& g, int grow, int col, float (&gate)[W], const float (&up)[W]) {
    uint4* o = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(g.c) + (int64_t)grow * g.n[0] + col);
#pragma unroll
    for (int i = 0; i < W; ++i) gate[i] = gate[i] / (1.f + __expf(-gate[i])) * up[i];
#pragma unroll
    for (int j = 0; j < W / 8; ++j) o[j] = pack8(gate + 8 * j);
}

// q/k/v: bias, rotary embedding with the pairing (i, i + d/2) at the row's position, bf16 store
// to the compact output and, for k/v, straight into the cache row (scatter fused).
// lo/hi: W columns of each rotary half; col: column of lo[0] inside segment seg; j0: its index
// inside the half head.
template <int W>
__device__ __forceinline__ void out_qkv(const GemmArgs& g, int grow, int pos, int seg, int col, int j0, float (&lo)[W],
                                        float (&hi)[W]) {
    const int half = g.head_dim >> 1;
    const __nv_bfloat16* bias = static_cast<const __nv_bfloat16*>(g.bias[seg]);
    if (bias) {
#pragma unroll
        for (int i = 0; i < W; ++i) {
            lo[i] += __bfloat162float(bias[col + i]);
            hi[i] += __bfloat162float(bias[col + half + i]);
        }
    }
    if (seg < g.rope_segments) {
        const int pp = pos < 0 ? 0 : pos;
        const float4* cs = reinterpret_cast<const float4*>(g.rope_cos + (int64_t)pp * half + j0);
        const float4* sn = reinterpret_cast<const float4*>(g.rope_sin + (int64_t)pp * half + j0);
#pragma unroll
        for (int j = 0; j < W / 4; ++j) {
            const float4 c4 = cs[j], s4 = sn[j];
            const float c[4] = {c4.x, c4.y, c4.z, c4.w}, sv[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float x = lo[4 * j + i], y = hi[4 * j + i];
                lo[4 * j + i] = x * c[i] - y * sv[i];
                hi[4 * j + i] = y * c[i] + x * sv[i];
            }
        }
    }
    const int nseg = g.n[seg];
    __nv_bfloat16* cache = seg == 1 ? static_cast<__nv_bfloat16*>(g.cache_k)
                         : seg == 2 ? static_cast<__nv_bfloat16*>(g.cache_v) : nullptr;
    int64_t orow = grow;
    bool o1_ok = g.out[seg] != nullptr;
    if (seg >= 1 && g.kv_out_rows && o1_ok) {          // the row's place in its request's private slot array
        const int r = __ldg(g.kv_out_rows + grow);
        if ((unsigned)r >= (unsigned)g.kv_out_stride) {
            atomicOr(g.status, kFlagBadIndex);
            o1_ok = false;
        }
        orow = (int64_t)(grow / g.rows_per_req) * g.kv_out_stride + r;
    }
    __nv_bfloat16* o1 = o1_ok ? static_cast<__nv_bfloat16*>(g.out[seg]) + orow * nseg + col : nullptr;
    __nv_bfloat16* o2 = (cache && pos >= 0)
                            ? cache + (int64_t)(grow / g.rows_per_req) * g.kv_batch_stride + (int64_t)pos * nseg + col
                            : nullptr;
#pragma unroll
    for (int j = 0; j < W / 8; ++j) {
        const uint4 l = pack8(lo + 8 * j), h = pack8(hi + 8 * j);
        if (o1) { reinterpret_cast<uint4*>(o1)[j] = l; reinterpret_cast<uint4*>(o1 + half)[j] = h; }
        if (o2) { reinterpret_cast<uint4*>(o2)[j] = l; reinterpret_cast<uint4*>(o2 + half)[j] = h; }
    }
}

// Segment and in-segment column of the 128-wide column unit u128 of a q/k/v projection.
__device__ __forceinline__ void qkv_unit(const GemmArgs& g, int u128, int& seg, int& c0) {
    seg = 0; c0 = u128 * 128;
    while (seg < 2 && c0 >= g.n[seg]) { c0 -= g.n[seg]; ++seg; }
}

// ---- split tiles: partial slots and their ordered sum -------------------------------------------
// A tile whose K range is cut between CTAs is accumulated through fp32 partial tiles.  Each CTA owns
// two slots: slot 0 for its first segment, slot 1 for its last (segments in between are whole tiles
// and never need one).  Tile t's contributors are CTAs c_first..c_last; CTA c's part of it is that
// CTA's first segment exactly when the CTA starts inside the tile.
// In the two-SM kernel's stream-K mode the contributors are clusters, the tile that is cut is the
// 256-row pair tile tp = nt * m_pairs + mt / 2, and each CTA of a cluster (rank = mt & 1) has its own
// pair of slots: slot = (cluster * 2 + segment) * 2 + rank.
__device__ __forceinline__ void tile_cover(const TcPlan& p, int t, int& c_first, int& c_last) {
    if (p.pair_u) {
        const int nt = t / p.m_tiles, mt = t - nt * p.m_tiles;
        t = nt * p.m_pairs + (mt >> 1);
    }
    const int U = p.pair_u ? p.pair_u : p.U;
    c_first = (int)(((int64_t)t * p.KB) / U);
    c_last = (int)(((int64_t)(t + 1) * p.KB - 1) / U);
}
__device__ __forceinline__ int64_t slot_of(const TcPlan& p, int t, int c) {
    if (p.pair_u) {
        const int nt = t / p.m_tiles, mt = t - nt * p.m_tiles;
        const int tp = nt * p.m_pairs + (mt >> 1);
        return ((int64_t)c * 2 + ((int64_t)c * p.pair_u >= (int64_t)tp * p.KB ? 0 : 1)) * 2 + (mt & 1);
    }
    return (int64_t)c * 2 + ((int64_t)c * p.U >= (int64_t)t * p.KB ? 0 : 1);
}

// Ordered sums over the contributing CTAs' partial tiles of one row for 16 adjacent columns
// starting at column group pc0 and, if pc1 >= 0, 16 more starting at pc1.  Loads are issued two
// CTAs at a time for all eight column groups (16 independent 16-byte loads in flight per thread)
// and added in ascending CTA order, which keeps the result bitwise reproducible.
template <int NC>      // contributing CTAs per round of loads: 2, or 4 where the kernel may use 255 registers
__device__ __forceinline__ void sum_slots16(const float* __restrict__ partial, const TcPlan& p, int t, int c_first,
                                            int c_last, int pc0, int pc1, int row, float (&lo)[16], float (&hi)[16]) {
#pragma unroll
    for (int i = 0; i < 16; ++i) { lo[i] = 0.f; hi[i] = 0.f; }
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    const int o0 = pc0 * TC_BM + row, o1 = (pc1 < 0 ? pc0 : pc1) * TC_BM + row;
    for (int c = c_first; c <= c_last; c += NC) {
        float4 a[NC][4], b[NC][4];
#pragma unroll
        for (int i = 0; i < NC; ++i) {
            const bool in = c + i <= c_last;
            const float4* src = reinterpret_cast<const float4*>(partial) + slot_of(p, t, in ? c + i : c) * (TC_SLOT_FLOATS / 4);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                a[i][j] = in ? __ldcg(src + o0 + j * TC_BM) : zero;
                b[i][j] = (in && pc1 >= 0) ? __ldcg(src + o1 + j * TC_BM) : zero;
            }
        }
#pragma unroll
        for (int i = 0; i < NC; ++i) {
            if (c + i <= c_last) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    lo[4 * j] += a[i][j].x; lo[4 * j + 1] += a[i][j].y; lo[4 * j + 2] += a[i][j].z; lo[4 * j + 3] += a[i][j].w;
                    hi[4 * j] += b[i][j].x; hi[4 * j + 1] += b[i][j].y; hi[4 * j + 2] += b[i][j].z; hi[4 * j + 3] += b[i][j].w;
                }
            }
        }
    }
}

// Softmax statistics of W logits starting at vocabulary index col: running (max, sum exp(z - max),
// arg max with the lowest index on ties).
template <int W>
__device__ __forceinline__ void logit_stats_update(const float (&v)[W], int col, float& m, float& s, int& arg) {
    float cm = v[0];
    int ca = 0;
#pragma unroll
    for (int i = 1; i < W; ++i)
        if (v[i] > cm) { cm = v[i]; ca = i; }
    if (cm > m) {
        s *= __expf(m - cm);
        m = cm;
        arg = col + ca;
    }
#pragma unroll
    for (int i = 0; i < W; ++i) s += __expf(v[i] - m);
}

// The same for one group of 16 columns, four CTAs at a time (the registers the second group would take hold
// two more CTAs' loads): epilogues without a second group (residual, logits) have nine or ten contributors per
// tile on the narrow projections, and every round of loads is a trip to L2.
__device__ __forceinline__ void sum_slots16_single(const float* __restrict__ partial, const TcPlan& p, int t, int c_first,
                                                   int c_last, int pc0, int row, float (&lo)[16]) {
#pragma unroll
    for (int i = 0; i < 16; ++i) lo[i] = 0.f;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    const int o0 = pc0 * TC_BM + row;
    for (int c = c_first; c <= c_last; c += 4) {
        float4 a[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const bool in = c + i <= c_last;
            const float4* src = reinterpret_cast<const float4*>(partial) + slot_of(p, t, in ? c + i : c) * (TC_SLOT_FLOATS / 4);
#pragma unroll
            for (int j = 0; j < 4; ++j) a[i][j] = in ? __ldcg(src + o0 + j * TC_BM) : zero;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (c + i <= c_last) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    lo[4 * j] += a[i][j].x; lo[4 * j + 1] += a[i][j].y; lo[4 * j + 2] += a[i][j].z; lo[4 * j + 3] += a[i][j].w;
                }
            }
        }
    }
}

// Work items of the finish per output tile: 16 output columns each (q/k/v: 16 of each rotary half).
__host__ __device__ __forceinline__ int finish_items_per_tile(int epilogue) {
    return (epilogue == kEpiResidual || epilogue == kEpiLogits) ? 16 : 8;
}

// Finish of one work item of split tile t = nt * m_tiles + mt for tile row `row`.
// The row's 32 bytes of residual under an item's 16 columns (kEpiResidual).
__device__ __forceinline__ void load_residual16(const GemmArgs& g, int grow, int col, uint4 (&res)[2]) {
    const int64_t roff = g.resid_off ? __ldcg(g.resid_off + grow) : (int64_t)grow * g.n[0];
    const uint4* rp = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(g.resid) + roff + col);
    res[0] = __ldcg(rp); res[1] = __ldcg(rp + 1);
}

// Where an item of the finish lives: everything that can be worked out before the projection has finished.
struct FinishItem {
    int nt, grow, c_first, c_last, pc0, pc1, u128, lo_col;
    bool skip;
};
__device__ __forceinline__ FinishItem finish_plan(const GemmArgs& g, const TcPlan& p, int t, int item, int row) {
    FinishItem f;
    f.nt = t / p.m_tiles;
    f.grow = (t - f.nt * p.m_tiles) * TC_BM + row;
    tile_cover(p, t, f.c_first, f.c_last);
    const int half = g.head_dim >> 1;
    f.pc1 = -1; f.u128 = 0; f.lo_col = 0; f.skip = false;
    if (g.epilogue == kEpiResidual || g.epilogue == kEpiLogits) {
        f.pc0 = item * 4;
        if (g.epilogue == kEpiLogits && f.nt * 2 + (item >> 3) >= p.units) f.skip = true;   // past the vocabulary's end
    } else if (g.epilogue == kEpiSwiGLU) {
        f.pc0 = item * 4; f.pc1 = 32 + f.pc0;
    } else {
        const int h = item >> 2, r = item & 3;
        f.u128 = f.nt * 2 + h;
        if (f.u128 >= p.units) f.skip = true;                                 // the tile's second half is past the end
        f.lo_col = g.head_dim == 128 ? 16 * r : 64 * (r >> 1) + 16 * (r & 1);   // column inside the 128-wide unit
        f.pc0 = 32 * h + (f.lo_col >> 2);
        f.pc1 = f.pc0 + (half >> 2);
    }
    return f;
}

// res: the residual, loaded by the caller (kEpiResidual only).
template <int NC>
__device__ __forceinline__ void finish_item(const GemmArgs& g, const TcPlan& p, int t, int item, int row, const FinishItem& f,
                                            const uint4 (&res)[2]) {
    if (f.skip) return;
    const int nt = f.nt, grow = f.grow, c_first = f.c_first, c_last = f.c_last, pc0 = f.pc0, pc1 = f.pc1, u128 = f.u128,
              lo_col = f.lo_col;
    const int half = g.head_dim >> 1;
    int pos = 0;
    if (g.epilogue == kEpiQKV) pos = __ldcg(g.row_pos + grow);     // independent of the sums: overlaps their loads
    float lo[16], hi[16];
    if (pc1 < 0) sum_slots16_single(g.partial, p, t, c_first, c_last, pc0, row, lo);
    else sum_slots16<NC>(g.partial, p, t, c_first, c_last, pc0, pc1, row, lo, hi);
    if (g.epilogue == kEpiResidual) {
        const uint32_t rw[8] = {res[0].x, res[0].y, res[0].z, res[0].w, res[1].x, res[1].y, res[1].z, res[1].w};
#pragma unroll
        for (int i = 0; i < 8; ++i) { lo[2 * i] += bf16_lo(rw[i]); lo[2 * i + 1] += bf16_hi(rw[i]); }
        uint4* o = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(g.c) + (int64_t)grow * g.n[0] + nt * TC_BN + item * 16);
        o[0] = pack8(lo); o[1] = pack8(lo + 8);
    } else if (g.epilogue == kEpiLogits) {
        float m = -INFINITY, sm = 0.f;
        int arg = 0;
        logit_stats_update<16>(lo, nt * TC_BN + item * 16, m, sm, arg);
        g.logit_stats[((int64_t)grow * p.n_tiles + nt) * 16 + item] = make_float4(m, sm, __int_as_float(arg), 0.f);
    } else if (g.epilogue == kEpiSwiGLU) {
        out_swiglu<16>(g, grow, nt * 128 + item * 16, lo, hi);
    } else {
        int seg, c0;
        qkv_unit(g, u128, seg, c0);
        out_qkv<16>(g, grow, pos, seg, c0 + lo_col, lo_col & (half - 1), lo, hi);
    }
}

// Epilogue of a whole tile straight from TMEM (the CTA covered the tile's entire K range):
// thread = one row of the tile, 32 accumulator columns per tcgen05.ld.
__device__ __forceinline__ void direct_epilogue(const GemmArgs& g, const TcPlan& p, uint32_t taddr, int nt, int grow,
                                                bool valid, int nchunks) {
    if (g.epilogue == kEpiResidual) {
        for (int c = 0; c < nchunks; ++c) {
            float v[32];
            tc_ld32(taddr + c * 32, v);
            if (valid) out_residual<32>(g, grow, nt * TC_BN + c * 32, v);
        }
    } else if (g.epilogue == kEpiLogits) {
        float m = -INFINITY, sm = 0.f;
        int arg = 0;
        for (int c = 0; c < nchunks; ++c) {
            float v[32];
            tc_ld32(taddr + c * 32, v);
            logit_stats_update<32>(v, nt * TC_BN + c * 32, m, sm, arg);
        }
        if (valid) g.logit_stats[((int64_t)grow * p.n_tiles + nt) * 16] = make_float4(m, sm, __int_as_float(arg), 0.f);
    } else if (g.epilogue == kEpiSwiGLU) {
        for (int c = 0; c < 4; ++c) {
            float gate[32], up[32];
            tc_ld32(taddr + c * 32, gate);
            tc_ld32(taddr + 128 + c * 32, up);
            if (valid) out_swiglu<32>(g, grow, nt * 128 + c * 32, gate, up);
        }
    } else {
        const int half = g.head_dim >> 1;
        const int pos = valid ? __ldcg(g.row_pos + grow) : 0;
        for (int h = 0; h < nchunks / 4; ++h) {
            int seg, c0;
            qkv_unit(g, nt * 2 + h, seg, c0);
            for (int r = 0; r < 2; ++r) {
                // d = 128: chunks (r, r + 2) of the unit; d = 64: chunks (2r, 2r + 1)
                const int cl = g.head_dim == 128 ? r : 2 * r, ch = g.head_dim == 128 ? r + 2 : 2 * r + 1;
                float lo[32], hi[32];
                tc_ld32(taddr + h * 128 + cl * 32, lo);
                tc_ld32(taddr + h * 128 + ch * 32, hi);
                if (valid) out_qkv<32>(g, grow, pos, seg, c0 + cl * 32, (cl * 32) & (half - 1), lo, hi);
            }
        }
    }
}

// Where row `row` of the A operand comes from (element offset inside rp.x); `writer` (one thread per
// row) records the row's position and source for the later kernels and raises the bad-index flag.
__device__ __forceinline__ int64_t prep_row_source(const GemmArgs& g, int row, bool writer) {
    const RowPrep& rp = g.prep;
    const int rows_per_req = rp.k + rp.e;
    int64_t src = (int64_t)row * g.K;
    if (rp.enabled == 3) {       // compact rows picked by index
        const int b = row / rows_per_req;
        const int ci = rp.compact_idx[row];
        if (ci < 0 || ci >= rp.compact_rows) {
            if (writer) atomicOr(g.status, kFlagBadIndex);
        }
        src = ((int64_t)b * rp.compact_rows + (ci < 0 || ci >= rp.compact_rows ? 0 : ci)) * g.K;
    }
    if (rp.enabled == 1) {       // rows of R: position from the anchor / extra-row lists
        const int b = row / rows_per_req, i = row - b * rows_per_req;
        const int pos = row_position(rp.anchor_idx, rp.k, rp.extra_rows, rp.e, b, i, rp.affix_start,
                                     rp.affix_len, rp.ctx_len);
        if (!rp.x_is_compact) {
            if (rp.token_ids) {       // x is an embedding table: the row of the token at that position
                int id = rp.token_ids[(int64_t)b * rp.ctx_len + (pos < 0 ? 0 : pos)];
                if (id < 0 || id >= rp.table_rows) {
                    if (writer) atomicOr(g.status, kFlagBadIndex);
                    id = 0;
                }
                src = (int64_t)id * g.K;
            } else {
                src = (int64_t)b * rp.x_batch_stride + (int64_t)(pos < 0 ? 0 : pos) * g.K;
            }
        } else if (rp.compact_idx) {
            const int ci = rp.compact_idx[row];
            src = ((int64_t)b * rp.compact_rows + (ci < 0 ? 0 : ci)) * g.K;
        }
        if (writer) {
            rp.row_pos[row] = pos;
            rp.row_src[row] = src;
            if (pos < 0) atomicOr(g.status, kFlagBadIndex);
        }
    }
    return src;
}

// out = bf16(x * rsqrt(mean(x^2) + eps) * g) for one row, by one warp: rows of up to 4096 values in one pass from
// registers; longer ones in two passes with eight independent 16-byte loads in flight per lane (the second pass hits
// L1 / L2).
__device__ __forceinline__ void rmsnorm_row_warp(const uint4* __restrict__ xr, const uint4* __restrict__ gn,
                                                 uint4* __restrict__ out, int hidden, float eps, int lane,
                                                 uint4* __restrict__ raw) {
    const int nchunk = hidden >> 3;
    if (nchunk <= 512) {
        // rows of up to 4096 values: one pass, the row stays in registers (sixteen 16-byte loads in flight per lane,
        // one trip to memory per row instead of two), the gain is requested before the warp-wide sum
        uint4 u[16];
        float s1 = 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int c = i * 32 + lane;
            u[i] = c < nchunk ? __ldcg(xr + c) : make_uint4(0, 0, 0, 0);
        }
        if (raw) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int c = i * 32 + lane;
                if (c < nchunk) raw[c] = u[i];
            }
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) { const float a = bf16_lo(w[e]), b = bf16_hi(w[e]); s1 += a * a + b * b; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s1 += __shfl_xor_sync(0xffffffffu, s1, o);
        const float rstd1 = rsqrtf(s1 / (float)hidden + eps);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int c = i * 32 + lane;
            if (c < nchunk) {
                const uint4 gg = __ldg(gn + c);
                const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
                const uint32_t gw[4] = {gg.x, gg.y, gg.z, gg.w};
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
    for (int c0 = 0; c0 < nchunk; c0 += 256) {
        uint4 u[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int c = c0 + i * 32 + lane;
            u[i] = c < nchunk ? __ldcg(xr + c) : make_uint4(0, 0, 0, 0);
            if (raw && c < nchunk) raw[c] = u[i];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) { const float a = bf16_lo(w[e]), b = bf16_hi(w[e]); ss += a * a + b * b; }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float rstd = rsqrtf(ss / (float)hidden + eps);
    for (int c0 = 0; c0 < nchunk; c0 += 256) {
        uint4 u[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int c = c0 + i * 32 + lane;
            u[i] = c < nchunk ? __ldcg(xr + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int c = c0 + i * 32 + lane;
            if (c < nchunk) {
                const uint4 gg = __ldg(gn + c);
                const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
                const uint32_t gw[4] = {gg.x, gg.y, gg.z, gg.w};
                uint32_t r[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    r[e] = pack_bf16(bf16_lo(w[e]) * rstd * bf16_lo(gw[e]), bf16_hi(w[e]) * rstd * bf16_hi(gw[e]));
                out[c] = make_uint4(r[0], r[1], r[2], r[3]);
            }
        }
    }
}

// Phase 0 of the projection kernels: the rows of R (or compact rows) -> RMSNorm -> the A operand,
// then a grid-wide barrier; the rows are read back through TMA.  With no more rows than CTAs a
// whole CTA takes a row (shortest latency); with many rows every warp takes rows of its own, which
// keeps six rows in flight per SM instead of one.
__device__ __forceinline__ void prep_phase(const GemmArgs& g, float* red, volatile int* abort_flag, unsigned int& nbar) {
    const RowPrep& rp = g.prep;
    const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(rp.x);
    __nv_bfloat16* a_out = static_cast<__nv_bfloat16*>(const_cast<void*>(g.a));
    __nv_bfloat16* raw = static_cast<__nv_bfloat16*>(rp.raw_out);
    if (g.M <= (int)gridDim.x) {
        for (int row = blockIdx.x; row < g.M; row += gridDim.x) {
            const int64_t src = prep_row_source(g, row, threadIdx.x == 0);
            rmsnorm_row(reinterpret_cast<const uint4*>(x + src), reinterpret_cast<const uint4*>(rp.gain),
                        reinterpret_cast<uint4*>(a_out + (int64_t)row * g.K), g.K, rp.eps, red,
                        raw ? reinterpret_cast<uint4*>(raw + (int64_t)row * g.K) : nullptr);
        }
    } else {
        const int nw = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        // the source of the next row (index lookups: a dependent trip to memory) is asked for before this row is read
        int row = blockIdx.x * nw + warp;
        int64_t src = row < g.M ? prep_row_source(g, row, lane == 0) : 0;
        while (row < g.M) {
            const int next = row + gridDim.x * nw;
            const int64_t src_next = next < g.M ? prep_row_source(g, next, lane == 0) : 0;
            rmsnorm_row_warp(reinterpret_cast<const uint4*>(x + src), reinterpret_cast<const uint4*>(rp.gain),
                             reinterpret_cast<uint4*>(a_out + (int64_t)row * g.K), g.K, rp.eps, lane,
                             raw ? reinterpret_cast<uint4*>(raw + (int64_t)row * g.K) : nullptr);
            row = next;
            src = src_next;
        }
    }
    asm volatile("fence.proxy.async;" ::: "memory");   // the rows are read back through TMA
    grid_barrier(g.grid_bar, ++nbar, abort_flag, g.debug_expire != 0);
    asm volatile("fence.proxy.async;" ::: "memory");
}

// The same row preparation as a kernel of its own, for many rows: inside the projection kernel only the CTA's six warps
// work on it (one CTA per SM: 14 752 rows took 88-95 us per launch, 2.5 TB/s); here sixteen warps per SM do, and the
// projection starts without the grid-wide barrier.
__global__ void __launch_bounds__(256, 2) prep_rows_kernel(const GemmArgs g) {
    pdl_wait();
    pdl_launch_dependents();
    const RowPrep& rp = g.prep;
    const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(rp.x);
    __nv_bfloat16* a_out = static_cast<__nv_bfloat16*>(const_cast<void*>(g.a));
    __nv_bfloat16* raw = static_cast<__nv_bfloat16*>(rp.raw_out);
    const int nw = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int row = blockIdx.x * nw + warp;
    int64_t src = row < g.M ? prep_row_source(g, row, lane == 0) : 0;
    while (row < g.M) {
        const int next = row + gridDim.x * nw;
        const int64_t src_next = next < g.M ? prep_row_source(g, next, lane == 0) : 0;
        rmsnorm_row_warp(reinterpret_cast<const uint4*>(x + src), reinterpret_cast<const uint4*>(rp.gain),
                         reinterpret_cast<uint4*>(a_out + (int64_t)row * g.K), g.K, rp.eps, lane,
                         raw ? reinterpret_cast<uint4*>(raw + (int64_t)row * g.K) : nullptr);
        row = next;
        src = src_next;
    }
}

__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const GemmArgs g, const TcPlan p, const __grid_constant__ CUtensorMap mapA,
               const __grid_constant__ CUtensorMap mapB0, const __grid_constant__ CUtensorMap mapB1,
               const __grid_constant__ CUtensorMap mapB2) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ float red[TC_THREADS / 32];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + TC_STAGES * TC_STAGE_BYTES;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + TC_STAGES * TC_STAGE_BYTES + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + TC_STAGES * TC_STAGE_BYTES + 200);
    auto full_bar = [&](int s) { return bars + 8 * s; };
    auto empty_bar = [&](int s) { return bars + 8 * (TC_STAGES + s); };
    auto tfull_bar = [&](int i) { return bars + 8 * (2 * TC_STAGES + i); };
    auto tempty_bar = [&](int i) { return bars + 8 * (2 * TC_STAGES + 2 + i); };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned int nbar = 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(tfull_bar(i), 1); mbar_init(tempty_bar(i), 4); }
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
    const int it0 = blockIdx.x * p.U;
    const int it1 = min(it0 + p.U, p.tiles * p.KB);
    // The weights are constant inputs (no earlier kernel writes them), so their loads may start
    // before the previous kernel has finished: fill the ring's weight halves now and ask L2 for the
    // k-blocks after that.  The activation halves follow once the producer kernel is done.
    const int kPrefetchL2 = p.prefetch;
    int prefilled = 0;
    if (warp == 0 && lane == 0) {
        const CUtensorMap* maps[3] = {&mapB0, &mapB1, &mapB2};
        const uint64_t pol_w = g.keep_weights ? policy_evict_last() : policy_evict_first();
        for (int i = 0; i < p.prefill + kPrefetchL2 && it0 + i < it1; ++i) {
            const int it = it0 + i, t = it / p.KB, kb = it - t * p.KB, nt = t / p.m_tiles;
            int row0, row1;
            const int s0 = half_source(g, p, nt, 0, row0), s1 = half_source(g, p, nt, 1, row1);
            if (i < p.prefill) {
                const uint32_t sB = base + i * TC_STAGE_BYTES + TC_A_BYTES;
                mbar_expect_tx(full_bar(i), TC_A_BYTES + TC_HALF_BYTES * (1 + (s1 >= 0)));
                tma_load_2d(sB, maps[s0], kb * TC_BK, row0, full_bar(i), pol_w);
                if (s1 >= 0) tma_load_2d(sB + TC_HALF_BYTES, maps[s1], kb * TC_BK, row1, full_bar(i), pol_w);
                prefilled = i + 1;
            } else {
                tma_prefetch_2d(maps[s0], kb * TC_BK, row0);
                if (s1 >= 0) tma_prefetch_2d(maps[s1], kb * TC_BK, row1);
            }
        }
    }
    // everything above overlaps the previous kernel's tail; its outputs are touched only below
    pdl_wait();
    pdl_launch_dependents();

    // ---------------- phase 0: gather the rows of R and RMSNorm them into A ----------------
    if (g.prep.enabled) prep_phase(g, red, abort_flag, nbar);

    // ---------------- phase 1: the contraction ----------------

    if (warp == 0 && lane == 0) {
        // TMA producer
        const CUtensorMap* maps[3] = {&mapB0, &mapB1, &mapB2};
        int stage = 0;
        uint32_t phase = 0;
        bool ok = !*abort_flag;
        const uint64_t pol_a = policy_evict_last(), pol_w = g.keep_weights ? pol_a : policy_evict_first();
        for (int it = it0; it < it1 && ok;) {
            const int t = it / p.KB, kb0 = it - t * p.KB;
            const int kb1 = min(p.KB, kb0 + (it1 - it));
            const int nt = t / p.m_tiles, mt = t - nt * p.m_tiles;
            int row0, row1;
            const int s0 = half_source(g, p, nt, 0, row0), s1 = half_source(g, p, nt, 1, row1);
            const uint32_t bytes = TC_A_BYTES + TC_HALF_BYTES * (1 + (s1 >= 0));
            for (int kb = kb0; kb < kb1; ++kb) {
                const uint32_t sA = base + stage * TC_STAGE_BYTES, sB = sA + TC_A_BYTES;
                if (prefilled > 0) {          // this stage's weight halves are already on their way
                    --prefilled;
                    tma_load_2d(sA, &mapA, kb * TC_BK, mt * TC_BM, full_bar(stage), pol_a);
                } else {
                    if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1, abort_flag))) break;
                    mbar_expect_tx(full_bar(stage), bytes);
                    tma_load_2d(sA, &mapA, kb * TC_BK, mt * TC_BM, full_bar(stage), pol_a);
                    tma_load_2d(sB, maps[s0], kb * TC_BK, row0, full_bar(stage), pol_w);
                    if (s1 >= 0) tma_load_2d(sB + TC_HALF_BYTES, maps[s1], kb * TC_BK, row1, full_bar(stage), pol_w);
                }
                if (++stage == TC_STAGES) { stage = 0; phase ^= 1; }
            }
            it += kb1 - kb0;
        }
    } else if (warp == 1 && lane == 0) {
        // MMA issuer
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ok = !*abort_flag;
        for (int it = it0; it < it1 && ok;) {
            const int t = it / p.KB, kb0 = it - t * p.KB;
            const int kb1 = min(p.KB, kb0 + (it1 - it));
            const int nt = t / p.m_tiles;
            int row1;
            const uint32_t idesc = idesc_bf16(half_source(g, p, nt, 1, row1) >= 0 ? 256 : 128);
            if (!(ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1, abort_flag))) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * TC_BN;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag))) break;
                tc_fence_after();
                const uint32_t sA = base + stage * TC_STAGE_BYTES, sB = sA + TC_A_BYTES;
                const uint64_t da = smem_desc_sw128(sA), db = smem_desc_sw128(sB);
#pragma unroll
                for (int k = 0; k < TC_BK / 16; ++k)
                    tc_mma(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                tc_commit(empty_bar(stage));      // the stage is free once these MMAs have read it
                if (++stage == TC_STAGES) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            tc_commit(tfull_bar(acc));            // accumulator complete
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            it += kb1 - kb0;
        }
    } else if (warp >= 2 && warp < 6) {
        // drain: whole tiles get their epilogue straight from TMEM; a tile whose K range is split
        // between CTAs goes to this CTA's fp32 partial slot, layout [column / 4][row][4]
        const int q = warp & 3;                   // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = !*abort_flag;
        const uint64_t pol_p = policy_evict_last();
        for (int it = it0; it < it1 && ok;) {
            const int t = it / p.KB, kb0 = it - t * p.KB;
            const int kb1 = min(p.KB, kb0 + (it1 - it));
            const int nt = t / p.m_tiles, mt = t - nt * p.m_tiles;
            int row1;
            const int nchunks = half_source(g, p, nt, 1, row1) >= 0 ? 8 : 4;
            if (!(ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag))) break;
            tc_fence_after();
            const bool valid = mt * TC_BM + row < g.M;
            const uint32_t taddr = tmem_base + acc * TC_BN + ((uint32_t)(q * 32) << 16);
            if (kb0 == 0 && kb1 == p.KB) {
                direct_epilogue(g, p, taddr, nt, mt * TC_BM + row, valid, nchunks);
            } else {
                float4* dst = reinterpret_cast<float4*>(g.partial) +
                              ((int64_t)blockIdx.x * 2 + (it == it0 ? 0 : 1)) * (TC_SLOT_FLOATS / 4);
                for (int c = 0; c < nchunks; ++c) {
                    float v[32];
                    tc_ld32(taddr + c * 32, v);
                    if (valid) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            st_hint_f4(&dst[(c * 8 + i) * TC_BM + row], make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]), pol_p);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            it += kb1 - kb0;
        }
    }
    tc_fence_before();
    __syncthreads();
    // ---------------- teardown ----------------
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) {
            atomicOr(g.status, kFlagWaitExpired);
            // Ring stages whose weight halves were requested before the dependency wait but whose activation tile
            // never was (the wait that ran out came first): send that tile now, so that the stage's full barrier
            // completes exactly when all of its copies have landed, and wait for it.  No copy may still be on its
            // way into this CTA's shared memory when the CTA returns.
            const uint64_t pol = policy_evict_last();
            for (int i = 0; i < prefilled; ++i)
                tma_load_2d(base + i * TC_STAGE_BYTES, &mapA, 0, 0, full_bar(i), pol);
            for (int i = 0; i < prefilled; ++i)
                for (uint32_t n = 0; n < TC_WAIT_LIMIT && !mbar_try_wait(full_bar(i), 0); ++n) __nanosleep(40);
            for (int i = 0; i < 4096; ++i) __nanosleep(64);   // copies of stages that were complete when a role gave up
        }
        __syncthreads();
    } else if (threadIdx.x == 0 && nbar > 0) {
        // the last CTA to leave re-arms the barrier words for the next launch
        __threadfence();
        if (atomicAdd(&g.grid_bar[1], 1u) == gridDim.x - 1) {
            g.grid_bar[0] = 0u;
            __threadfence();
            g.grid_bar[1] = 0u;
        }
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

// ---- cta_group::2: two SMs on one 256 x 256 output tile (many-row problems) -----------------------
// A cluster of two CTAs owns a tile: CTA r holds rows [128 r, 128 r + 128) of A and the r-th
// 128-row half of the weight tile in its own shared memory, so each SM moves half of the weight
// bytes per flop that the one-CTA kernel moves; the leader CTA's MMA thread issues
// tcgen05.mma.cta_group::2 (M = 256) and each CTA's TMEM receives its 128 rows of the result.
// Tiles are whole (no K split): clusters walk the tile list round-robin, weight-tile-major.
// Barriers: the leader's full[s] counts both CTAs' TMA bytes (announced by the leader's producer); empty[s] and tmem_full[a] live in
// each CTA and are signalled by a tcgen05.commit multicast to both; the leader's tmem_empty[a]
// collects the drain warps of both CTAs.
constexpr int TC2_STAGES = 6;
constexpr int TC2_STAGE_BYTES = TC_A_BYTES + TC_HALF_BYTES;     // 32 KB per CTA and stage
constexpr int TC2_SMEM = TC2_STAGES * TC2_STAGE_BYTES + 1024 + 256;

// Tile order of the two-SM kernel: groups of kTileGroupN weight tiles; inside a group the row
// pairs are walked with the group's weight tiles innermost.  The ~74 clusters running at any
// moment then cover a few row pairs x the group's weight tiles, whose A and B blocks (tens of MB) stay in
// L2 while they are reused, instead of streaming the whole A matrix from HBM once per weight tile.
// With three or more row pairs the weight tiles are loaded with the evict-last policy like the rows: every row
// pair re-reads them, and with evict-first (right for the few-row launches, whose weights pass through once) they
// left L2 between two uses.  Measured on the 32-layer step of 14 752 rows per layer under the power cap: 209-216 ms
// -> 191-197 ms at a 100-150 MHz higher SM clock (gate/up moved 8.6 GB through HBM per launch for 0.5 GB of
// operands; the saved traffic is power the tensor cores get); groups of 16 weight tiles then beat 8 by 1-2 %
// (4, 24, 32, 48 are slower), and cutting the row pairs into L2-sized blocks as well changes nothing more.
constexpr int kTileGroupN = 16;
constexpr int kKeepWeightsFromPairs = 3;
constexpr int kPrepKernelRows = 4096;     // from this many rows the row preparation is a kernel of its own
__device__ __forceinline__ void tile_coords(int t, int m_pairs, int n_tiles, int group_n, int& nt, int& mp) {
    const int full = n_tiles / group_n, per_group = group_n * m_pairs;
    if (t < full * per_group) {
        const int grp = t / per_group, r = t - grp * per_group;
        mp = r / group_n;
        nt = grp * group_n + (r - mp * group_n);
    } else {
        const int r = t - full * per_group, gn = n_tiles - full * group_n;
        mp = r / gn;
        nt = full * group_n + (r - mp * gn);
    }
}

// TMA load into this CTA's shared memory that completes on a barrier of the CTA pair's leader
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cluster,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster), "l"(policy)
        : "memory");
}
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc2_kernel(const GemmArgs g, const TcPlan p, const int clusters, const __grid_constant__ CUtensorMap mapA,
                const __grid_constant__ CUtensorMap mapB0, const __grid_constant__ CUtensorMap mapB1,
                const __grid_constant__ CUtensorMap mapB2) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ float red[TC_THREADS / 32];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + TC2_STAGES * TC2_STAGE_BYTES;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + TC2_STAGES * TC2_STAGE_BYTES + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + TC2_STAGES * TC2_STAGE_BYTES + 200);
    auto full_bar = [&](int s) { return bars + 8 * s; };
    auto empty_bar = [&](int s) { return bars + 8 * (TC2_STAGES + s); };
    auto tfull_bar = [&](int i) { return bars + 8 * (2 * TC2_STAGES + i); };
    auto tempty_bar = [&](int i) { return bars + 8 * (2 * TC2_STAGES + 2 + i); };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1;
    unsigned int nbar = 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC2_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(tfull_bar(i), 1); mbar_init(tempty_bar(i), 8); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;"
                     ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();          // the peer's barriers are initialised before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();
    pdl_launch_dependents();

    if (g.prep.enabled) prep_phase(g, red, abort_flag, nbar);

    const int m_pairs = (p.m_tiles + 1) >> 1;
    const int tiles = m_pairs * p.n_tiles;

    if (warp == 0 && lane == 0) {
        // TMA producer of this CTA: its 128 rows of A and its half of the weight tile
        const CUtensorMap* maps[3] = {&mapB0, &mapB1, &mapB2};
        int stage = 0, issued = 0;
        uint32_t phase = 0;
        bool ok = !*abort_flag;
        const uint64_t pol_a = policy_evict_last();
        const uint64_t pol_w = (g.keep_weights || p.w_keep) ? pol_a : policy_evict_first();
        // work list: whole tiles round-robin (pair_u == 0), or this cluster's contiguous range of
        // (tile, K block) iterations, tiles in weight-tile-major order (stream-K)
        const long long it_end = p.pair_u ? min((long long)(cluster_id + 1) * p.pair_u, (long long)tiles * p.KB) : 0;
        long long it = p.pair_u ? (long long)cluster_id * p.pair_u : 0;
        for (int t = p.pair_u ? (int)(it / p.KB) : cluster_id; ok && (p.pair_u ? it < it_end : t < tiles);) {
            int nt, mp;
            if (p.pair_u) { nt = t / m_pairs; mp = t - nt * m_pairs; } else tile_coords(t, m_pairs, p.n_tiles, p.group_n, nt, mp);
            const int kb0 = p.pair_u ? (int)(it - (long long)t * p.KB) : 0;
            const int kb1 = p.pair_u ? (int)min((long long)p.KB, (long long)(kb0 + (it_end - it))) : p.KB;
            int brow;
            const int bs = half_source(g, p, nt, (int)rank, brow);
            const int arow = (mp * 2 + (int)rank) * TC_BM;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1, abort_flag))) break;
                const uint32_t sA = base + stage * TC2_STAGE_BYTES, sB = sA + TC_A_BYTES;
                const uint32_t lead_full = mapa_u32(full_bar(stage), 0);
                // the leader announces the bytes of both CTAs; the peer's copies only report completion
                if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * TC2_STAGE_BYTES);
                tma_load_2d_pair(sA, &mapA, kb * TC_BK, arow, lead_full, pol_a);
                tma_load_2d_pair(sB, maps[bs], kb * TC_BK, brow, lead_full, pol_w);
                ++issued;
                if (++stage == TC2_STAGES) { stage = 0; phase ^= 1; }
            }
            if (p.pair_u) { it += kb1 - kb0; ++t; } else t += clusters;
        }
        // wait until the MMAs have consumed everything this CTA loaded, so that no signal from the
        // leader can arrive after this CTA has left
        for (int i = 0; i < min(issued, TC2_STAGES) && ok; ++i) {
            ok = mbar_wait(empty_bar(stage), phase ^ 1, abort_flag);
            if (++stage == TC2_STAGES) { stage = 0; phase ^= 1; }
        }
    } else if (warp == 1 && lane == 0 && rank == 0) {
        // MMA issuer (leader CTA only)
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ok = !*abort_flag;
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
        const long long it_end = p.pair_u ? min((long long)(cluster_id + 1) * p.pair_u, (long long)tiles * p.KB) : 0;
        long long it = p.pair_u ? (long long)cluster_id * p.pair_u : 0;
        for (int t = p.pair_u ? (int)(it / p.KB) : cluster_id; ok && (p.pair_u ? it < it_end : t < tiles);) {
            const int kb0 = p.pair_u ? (int)(it - (long long)t * p.KB) : 0;
            const int kb1 = p.pair_u ? (int)min((long long)p.KB, (long long)(kb0 + (it_end - it))) : p.KB;
            if (!(ok = mbar_wait_cluster(tempty_bar(acc), acc_phase ^ 1, abort_flag))) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * TC_BN;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!(ok = mbar_wait_cluster(full_bar(stage), phase, abort_flag))) break;
                tc_fence_after();
                const uint32_t sA = base + stage * TC2_STAGE_BYTES, sB = sA + TC_A_BYTES;
                const uint64_t da = smem_desc_sw128(sA), db = smem_desc_sw128(sB);
#pragma unroll
                for (int k = 0; k < TC_BK / 16; ++k)
                    tc2_mma(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                tc2_commit_both(empty_bar(stage));
                if (++stage == TC2_STAGES) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            tc2_commit_both(tfull_bar(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            if (p.pair_u) { it += kb1 - kb0; ++t; } else t += clusters;
        }
    } else if (warp >= 2 && warp < 6) {
        // drain: this CTA's 128 rows of the tile, epilogue straight from TMEM
        const int q = warp & 3;
        const int row = q * 32 + lane;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = !*abort_flag;
        const long long it_end = p.pair_u ? min((long long)(cluster_id + 1) * p.pair_u, (long long)tiles * p.KB) : 0;
        long long it = p.pair_u ? (long long)cluster_id * p.pair_u : 0;
        const long long it_first = it;
        const uint64_t pol_p = policy_evict_last();
        for (int t = p.pair_u ? (int)(it / p.KB) : cluster_id; ok && (p.pair_u ? it < it_end : t < tiles);) {
            int nt, mp;
            if (p.pair_u) { nt = t / m_pairs; mp = t - nt * m_pairs; } else tile_coords(t, m_pairs, p.n_tiles, p.group_n, nt, mp);
            const int kb0 = p.pair_u ? (int)(it - (long long)t * p.KB) : 0;
            const int kb1 = p.pair_u ? (int)min((long long)p.KB, (long long)(kb0 + (it_end - it))) : p.KB;
            const int grow = (mp * 2 + (int)rank) * TC_BM + row;
            if (!(ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag))) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + acc * TC_BN + ((uint32_t)(q * 32) << 16);
            if (kb0 == 0 && kb1 == p.KB) {
                direct_epilogue(g, p, taddr, nt, grow, grow < g.M, 8);
            } else {
                // a tile whose K range is cut between clusters: this CTA's 128 rows to its fp32 partial slot
                float4* dst = reinterpret_cast<float4*>(g.partial) +
                              (((int64_t)cluster_id * 2 + (it == it_first ? 0 : 1)) * 2 + rank) * (TC_SLOT_FLOATS / 4);
                for (int c = 0; c < 8; ++c) {
                    float v[32];
                    tc_ld32(taddr + c * 32, v);
                    if (grow < g.M) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            st_hint_f4(&dst[(c * 8 + i) * TC_BM + row], make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]), pol_p);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_u32(tempty_bar(acc), 0));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            if (p.pair_u) { it += kb1 - kb0; ++t; } else t += clusters;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) {
            atomicOr(g.status, kFlagWaitExpired);
            for (int i = 0; i < 4096; ++i) __nanosleep(64);
        }
        __syncthreads();
    } else if (threadIdx.x == 0 && nbar > 0) {
        __threadfence();
        if (atomicAdd(&g.grid_bar[1], 1u) == gridDim.x - 1) {
            g.grid_bar[0] = 0u;
            __threadfence();
            g.grid_bar[1] = 0u;
        }
    }
    cluster_sync_all();          // neither CTA leaves while its peer may still signal it
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

// Finish of the split tiles: grid row y finishes tile split.tile[y]; blockIdx.x * 256 +
// threadIdx.x -> (item, row).
struct SplitTiles {
    int n;
    int tile[160];     // one per CTA boundary that cuts a tile (at most SM count - 1)
};

// NC = 4 (255 registers, one block per SM) serves finishes of at most one block per SM with two column groups per
// item: the masked rows' query projection has nine or ten contributors per tile and every round is a trip to L2.
template <int NC>
__global__ void __launch_bounds__(256, NC == 2 ? 2 : 1) gemm_finish_kernel(const GemmArgs g, const TcPlan p, const SplitTiles split) {
    const int t = split.tile[blockIdx.y];
    const int mt = t % p.m_tiles;
    const int rows_per = p.m_tiles == 1 ? ((g.M + 31) & ~31) : TC_BM;
    const int w = blockIdx.x * 256 + threadIdx.x;
    const int row = w % rows_per, item = w / rows_per;
    const bool active = item < finish_items_per_tile(g.epilogue) && mt * TC_BM + row < g.M;
    // The residual rows and their offsets are outputs of kernels that had completed before the projection
    // whose tiles are finished here passed its own dependency wait, and this kernel starts after that: they can
    // be requested while the projection is still running.
    uint4 res[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
    FinishItem f{};
    if (active) {
        f = finish_plan(g, p, t, item, row);
        if (g.epilogue == kEpiResidual) load_residual16(g, f.grow, f.nt * TC_BN + item * 16, res);
    }
    pdl_wait();
    pdl_launch_dependents();
    if (!active) return;
    finish_item<NC>(g, p, t, item, row, f, res);
}

// ---- predict and commit (Eq. 2-3): confidence and arg max per row, commit rule per request ------
struct LogitAcc { float m, s; int arg; };
__device__ __forceinline__ void logit_merge(LogitAcc& a, float m, float s, int arg) {
    if (s == 0.f) return;            // an empty entry
    if (m > a.m || (m == a.m && arg < a.arg && s > 0.f)) {
        a.s = a.s * __expf(a.m - m) + s;
        a.m = m;
        a.arg = arg;
    } else {
        a.s += s * __expf(m - a.m);
    }
}

// One CTA per row: merges the per-tile statistics (16 entries for a tile whose K range was split
// between CTAs, one otherwise) in a fixed order.
__global__ void __launch_bounds__(256) logit_reduce_kernel(const GemmArgs g, const TcPlan p, int32_t* __restrict__ token,
                                                           float* __restrict__ confidence) {
    __shared__ float sm_m[256], sm_s[256];
    __shared__ int sm_a[256];
    pdl_wait();
    pdl_launch_dependents();
    const int row = blockIdx.x, mt = row / TC_BM;
    LogitAcc a{-INFINITY, 0.f, 0x7fffffff};
    for (int nt = threadIdx.x; nt < p.n_tiles; nt += 256) {
        int c_first, c_last;
        tile_cover(p, nt * p.m_tiles + mt, c_first, c_last);
        const int n_entries = c_first == c_last ? 1 : 16;
        const float4* e = g.logit_stats + ((int64_t)row * p.n_tiles + nt) * 16;
        for (int i = 0; i < n_entries; ++i) {
            if (n_entries == 16 && nt * 2 + (i >> 3) >= p.units) break;
            const float4 v = __ldcg(e + i);
            logit_merge(a, v.x, v.y, __float_as_int(v.z));
        }
    }
    sm_m[threadIdx.x] = a.m; sm_s[threadIdx.x] = a.s; sm_a[threadIdx.x] = a.arg;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            LogitAcc x{sm_m[threadIdx.x], sm_s[threadIdx.x], sm_a[threadIdx.x]};
            logit_merge(x, sm_m[threadIdx.x + o], sm_s[threadIdx.x + o], sm_a[threadIdx.x + o]);
            sm_m[threadIdx.x] = x.m; sm_s[threadIdx.x] = x.s; sm_a[threadIdx.x] = x.arg;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        token[row] = sm_a[0];
        confidence[row] = 1.f / sm_s[0];       // softmax probability of the arg max
    }
}

// One warp per request: commit the rows above the threshold, or the single most confident row
// (lowest index on ties) if there is none.
__global__ void __launch_bounds__(32) commit_kernel(const float* __restrict__ confidence, int n_blk, float threshold,
                                                    int32_t* __restrict__ commit) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, lane = threadIdx.x;
    const float* c = confidence + (int64_t)b * n_blk;
    int32_t* out = commit + (int64_t)b * n_blk;
    int any = 0, best = 0x7fffffff;
    float bestc = -INFINITY;
    for (int i = lane; i < n_blk; i += 32) {
        const float v = __ldcg(c + i);
        const int f = v > threshold;
        out[i] = f;
        any |= f;
        if (v > bestc) { bestc = v; best = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        any |= __shfl_xor_sync(0xffffffffu, any, o);
        const float oc = __shfl_xor_sync(0xffffffffu, bestc, o);
        const int ob = __shfl_xor_sync(0xffffffffu, best, o);
        if (oc > bestc || (oc == bestc && ob < best)) { bestc = oc; best = ob; }
    }
    if (!any && lane == 0 && best < n_blk) out[best] = 1;
}

// ---- host side ------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
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

// bf16 [rows, cols] row-major, box = 128 rows x 64 cols, 128-byte swizzle, zero fill out of bounds.
struct MapKey { const void* ptr; int rows, cols; };
struct MapEntry { MapKey key; CUtensorMap map; };
constexpr int kMapCache = 1024;   // a 32-layer model has over 200 weight matrices
std::mutex g_map_mutex;
MapEntry g_maps[kMapCache];
int g_map_count = 0, g_map_next = 0;

// The pointer is only good until the next call (a miss may replace any entry): callers copy the map.
const CUtensorMap* get_map(const void* ptr, int rows, int cols) {
    for (int i = 0; i < g_map_count; ++i)
        if (g_maps[i].key.ptr == ptr && g_maps[i].key.rows == rows && g_maps[i].key.cols == cols) return &g_maps[i].map;
    EncodeTiledFn fn = encode_fn();
    if (!fn) return nullptr;
    MapEntry& e = g_maps[g_map_next];
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return nullptr;
    e.key = MapKey{ptr, rows, cols};
    g_map_next = (g_map_next + 1) % kMapCache;
    if (g_map_count < kMapCache) ++g_map_count;
    return &e.map;
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

TcPlan make_plan(int M, int K, int units, bool swiglu) {
    TcPlan p{};
    p.units = units;
    p.m_tiles = (M + TC_BM - 1) / TC_BM;
    p.n_tiles = swiglu ? units : (units + 1) / 2;
    p.KB = K / TC_BK;
    p.tiles = p.m_tiles * p.n_tiles;
    const int64_t total = (int64_t)p.tiles * p.KB;
    const int g = (int)(total < sm_count() ? total : sm_count());
    p.U = (int)((total + g - 1) / g);
    p.ctas = (int)((total + p.U - 1) / p.U);
    p.smax = 2;   // partial slots per CTA
    // K blocks past the ring asked into L2 before the dependency wait: none by default (measured at configuration 2:
    // 168.1 us per layer-step at 0, 170.1 at 12, 175.7 at 28: with neighbours this short the requests compete with the
    // stream that follows); GemmArgs::prefetch_blocks sets it per projection.  The ring itself is filled before the
    // wait (174.9 us per layer-step with no stage prefilled, 169.1 with two, 167.9-168.6 with three or four).
    p.prefetch = 0;
    p.prefill = TC_STAGES;
    return p;
}

}  // namespace

size_t gemm_partial_bytes(int M, int K, int n_total, bool swiglu) {
    (void)M; (void)K; (void)n_total; (void)swiglu;
    // two fp32 partial tiles per CTA, at most one CTA per SM, whatever the problem size
    return (size_t)sm_count() * 2 * TC_SLOT_FLOATS * sizeof(float);
}

int launch_predict_commit(const GemmArgs& g, int batch, int n_blk, float threshold, int32_t* token, float* confidence,
                          int32_t* commit, cudaStream_t stream) {
    if (g.M == 0) return 0;
    const TcPlan p = make_plan(g.M, g.K, g.n[0] / 128, false);
    if (launch_pdl(logit_reduce_kernel, dim3(g.M), dim3(256), 0, stream, g, p, token, confidence) != cudaSuccess) return -1;
    if (launch_pdl(commit_kernel, dim3(batch), dim3(32), 0, stream, (const float*)confidence, n_blk, threshold, commit) !=
        cudaSuccess)
        return -1;
    return 2;
}

static int launch_gemm_impl(const GemmArgs& g, cudaStream_t stream);

int launch_gemm(const GemmArgs& g, cudaStream_t stream) {
    if (g.M == 0) return 0;
    // many rows: the row preparation runs as a kernel of its own (ACACHE_GEMM_PREP_KERNEL_ROWS: from how many rows; 0: never)
    static const int prep_rows = [] { const char* e = getenv("ACACHE_GEMM_PREP_KERNEL_ROWS"); return e ? atoi(e) : kPrepKernelRows; }();
    if (g.prep.enabled && prep_rows > 0 && g.M >= prep_rows) {
        const int blocks = std::min((g.M + 7) / 8, sm_count() * 2);
        if (launch_pdl(prep_rows_kernel, dim3(blocks), dim3(256), 0, stream, g) != cudaSuccess) return -1;
        GemmArgs g2 = g;
        g2.prep.enabled = 0;
        const int nl = launch_gemm_impl(g2, stream);
        return nl < 0 ? nl : nl + 1;
    }
    return launch_gemm_impl(g, stream);
}

static int launch_gemm_impl(const GemmArgs& g, cudaStream_t stream) {
    const bool swiglu = g.epilogue == kEpiSwiGLU;
    const int n_total = swiglu ? g.n[0] : g.n[0] + g.n[1] + g.n[2];
    TcPlan p = make_plan(g.M, g.K, n_total / 128, swiglu);
    if (g.prefetch_blocks > 0) p.prefetch = g.prefetch_blocks;
    std::lock_guard<std::mutex> lock(g_map_mutex);
    CUtensorMap map_a, map_b[3];
    {
        const CUtensorMap* m = get_map(g.a, g.M, g.K);
        if (!m) return -1;
        map_a = *m;
    }
    bool have_b[3] = {false, false, false};
    for (int i = 0; i < 3; ++i)
        if (g.b[i]) {
            const CUtensorMap* m = get_map(g.b[i], swiglu ? g.n[0] : g.n[i], g.K);
            if (m) { map_b[i] = *m; have_b[i] = true; }
        }
    if (!have_b[0]) return -1;
    const CUtensorMap* mA = &map_a;
    const CUtensorMap* mB[3] = {&map_b[0], have_b[1] ? &map_b[1] : &map_b[0], have_b[2] ? &map_b[2] : &map_b[0]};
    static bool attr = false;
    if (!attr) {
        cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM);
        cudaFuncSetAttribute(gemm_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC2_SMEM);
        attr = true;
    }
    // Two or more row tiles: two SMs per 256 x 256 tile.  With many tiles per cluster every tile is whole
    // and the clusters walk them round-robin; with few, the (tile, K block) iterations are cut into equal
    // contiguous ranges, one per cluster (stream-K), and the cut tiles go through the finish kernel.
    static const int pair_min_tiles = [] { const char* e = getenv("ACACHE_GEMM_PAIR_MIN_MTILES"); return e ? atoi(e) : 2; }();
    if (p.m_tiles >= pair_min_tiles && g.epilogue != kEpiLogits && (p.units % 2 == 0 || swiglu) && sm_count() >= 2) {
        const int m_pairs = (p.m_tiles + 1) / 2;
        const int tiles = m_pairs * p.n_tiles;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(sm_count() / 2 * 2);
        cfg.blockDim = dim3(TC_THREADS);
        cfg.dynamicSmemBytes = TC2_SMEM;
        cfg.stream = stream;
        cudaLaunchAttribute at[2];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = 2;
        // all clusters must be resident at once (phase 0 ends in a grid-wide barrier)
        static int max_clusters = 0;
        if (!max_clusters) {
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, gemm_tc2_kernel, &cfg) != cudaSuccess || n <= 0) {
                (void)cudaGetLastError();
                n = -1;
            }
            max_clusters = n;
        }
        if (max_clusters < 1) goto single_cta;
        TcPlan pp = p;
        pp.m_pairs = m_pairs;
        static const int group_n = [] { const char* e = getenv("ACACHE_GEMM_GROUP_N"); return e && atoi(e) > 0 ? atoi(e) : kTileGroupN; }();
        pp.group_n = group_n;
        static const int w_keep_from = [] { const char* e = getenv("ACACHE_GEMM_WKEEP_PAIRS"); return e ? atoi(e) : kKeepWeightsFromPairs; }();
        int clusters = std::min(std::min(max_clusters, sm_count() / 2), tiles);
        // measured: cutting tiles pays (partial tiles + finish kernel included) up to about two thirds of a wave
        static const int stream_k_pct = [] { const char* e = getenv("ACACHE_GEMM_PAIR_STREAMK_PCT"); return e ? atoi(e) : 66; }();
        SplitTiles split{};
        if (tiles * 100 <= stream_k_pct * std::min(max_clusters, sm_count() / 2)) {
            const int64_t total = (int64_t)tiles * p.KB;
            clusters = (int)std::min<int64_t>(std::min(max_clusters, sm_count() / 2), total);
            pp.pair_u = (int)((total + clusters - 1) / clusters);
            clusters = (int)((total + pp.pair_u - 1) / pp.pair_u);
            // pair tiles cut by a boundary between two clusters: both of their 128-row tiles go to the finish
            int last = -1;
            for (int c = 1; c < clusters; ++c) {
                const int64_t cut = (int64_t)c * pp.pair_u;
                if (cut % p.KB == 0) continue;
                const int tp = (int)(cut / p.KB);
                if (tp == last) continue;
                last = tp;
                const int nt = tp / m_pairs, mp = tp - nt * m_pairs;
                for (int r = 0; r < 2; ++r)
                    if (mp * 2 + r < p.m_tiles && split.n < 160) split.tile[split.n++] = nt * p.m_tiles + mp * 2 + r;
            }
            if (split.n >= 159) { pp.pair_u = 0; split.n = 0; clusters = std::min(std::min(max_clusters, sm_count() / 2), tiles); }
        }
        pp.w_keep = (m_pairs >= w_keep_from && pp.pair_u == 0) ? 1 : 0;      // whole tiles, walked by three or more row pairs
        cfg.gridDim = dim3(clusters * 2);
        if (cudaLaunchKernelEx(&cfg, gemm_tc2_kernel, g, pp, clusters, *mA, *mB[0], *mB[1], *mB[2]) != cudaSuccess) return -1;
        if (split.n == 0) return 1;
        const int per_tile = finish_items_per_tile(g.epilogue) * TC_BM;
        if (launch_pdl(gemm_finish_kernel<2>, dim3((per_tile + 255) / 256, split.n), dim3(256), 0, stream, g, pp, split) != cudaSuccess)
            return -1;
        return 2;
    }
single_cta:
    // a plain launch: a cooperative one measured ~2.5 us slower and cannot overlap the previous
    // kernel's tail; the grid never exceeds the SM count at one CTA per SM and the barrier is bounded
    if (launch_pdl(gemm_tc_kernel, dim3(p.ctas), dim3(TC_THREADS), TC_SMEM, stream, g, p, *mA, *mB[0], *mB[1], *mB[2]) !=
        cudaSuccess)
        return -1;
    // tiles whose K range is cut by a boundary between two CTAs, each listed once
    SplitTiles split{};
    for (int c = 1; c < p.ctas && split.n < 160; ++c) {
        const int64_t cut = (int64_t)c * p.U;
        if (cut % p.KB == 0) continue;
        const int t = (int)(cut / p.KB);
        if (split.n == 0 || split.tile[split.n - 1] != t) split.tile[split.n++] = t;
    }
    if (split.n == 0) return 1;
    const int rows_per = p.m_tiles == 1 ? ((g.M + 31) & ~31) : TC_BM;
    const int per_tile = finish_items_per_tile(g.epilogue) * rows_per;
    const dim3 fgrid((per_tile + 255) / 256, split.n);
    const bool wide = g.epilogue == kEpiQKV && (int)(fgrid.x * fgrid.y) <= sm_count();
    if ((wide ? launch_pdl(gemm_finish_kernel<4>, fgrid, dim3(256), 0, stream, g, p, split)
              : launch_pdl(gemm_finish_kernel<2>, fgrid, dim3(256), 0, stream, g, p, split)) != cudaSuccess)
        return -1;
    return 2;
}

}  // namespace acache
