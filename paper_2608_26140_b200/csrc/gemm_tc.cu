// C[M, N] = A[M, K] * B[N, K]^T (bf16 in, fp32 accumulate) on the 5th-generation tensor
// cores for the projections of the selective recomputation (Section 3.3).
//
// Design for a weight-streaming GEMM with few rows (M = K anchors + request rows, often
// <= 128) on 148 SMs:
//   * work = (output tiles of 128 x 256) x (K blocks of 64); the flat list of
//     (tile, k-block) iterations is cut into equal contiguous ranges, one per CTA, so every
//     SM streams the same number of weight bytes whatever N and K are;
//   * per CTA: one thread issues TMA loads of the A tile and the two 128-row halves of the
//     B tile into a 4-stage shared-memory ring (128-byte swizzle), one thread issues
//     tcgen05.mma (128 x 256 x 16) into a TMEM accumulator (two accumulators of 256 columns,
//     so the next segment's MMAs overlap the previous segment's drain), four warps drain
//     TMEM with tcgen05.ld and write fp32 partial tiles;
//   * a second kernel sums the partial tiles of each output tile in a fixed order
//     (bitwise reproducible) and applies the epilogue (gemm_epilogue.cuh).
// Every mbarrier wait is bounded: on expiry the CTA raises kFlagWaitExpired in the status
// word, stops issuing work, frees its TMEM and returns.
#include <cuda.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "gemm_epilogue.cuh"
#include "kernels.h"
#include "launch.h"

namespace acache {

constexpr int TC_BM = 128, TC_BN = 256, TC_BK = 64, TC_STAGES = 4;
constexpr int TC_A_BYTES = TC_BM * TC_BK * 2;          // 16 KB
constexpr int TC_HALF_BYTES = 128 * TC_BK * 2;         // 16 KB: one 128-row half of the B tile
constexpr int TC_STAGE_BYTES = TC_A_BYTES + 2 * TC_HALF_BYTES;
constexpr int TC_THREADS = 192;                        // warp 0: TMA, warp 1: MMA, warps 2-5: drain
constexpr int TC_SMEM = TC_STAGES * TC_STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int TC_SLOT_FLOATS = TC_BM * TC_BN;          // one fp32 partial tile
constexpr uint32_t TC_WAIT_LIMIT = 1u << 22;

struct TcPlan {
    int m_tiles, n_tiles, KB, tiles, U, ctas, smax;
    int units;            // 128-row B halves over all segments (non-SwiGLU) or ffn/128 (SwiGLU)
};

struct TcArgs {
    int M;
    int swiglu;
    int n[3];             // segment widths (non-SwiGLU)
    TcPlan p;
    float* partial;
    uint32_t* status;
};

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < TC_WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 128) {
            __nanosleep(40);
            if (*abort_flag) return false;
        }
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128 bytes with the
// 128-byte swizzle: 8-row groups are 1024 bytes apart; descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;                 // leading byte offset (ignored for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                 // descriptor version
    d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
    return d;
}
// Instruction descriptor: D fp32, A/B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t idesc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

// Which weight matrix and row the 128-row half `h` of N tile `nt` starts at; -1 if past the end.
__device__ __forceinline__ int half_source(const TcArgs& a, int nt, int h, int& row) {
    if (a.swiglu) {
        row = nt * 128;
        return h;                      // half 0: gate rows, half 1: up rows
    }
    int u = nt * 2 + h;
    if (u >= a.p.units) return -1;
    int r = u * 128, seg = 0;
    while (seg < 2 && r >= a.n[seg]) { r -= a.n[seg]; ++seg; }
    row = r;
    return seg;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const TcArgs a, const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB0,
               const __grid_constant__ CUtensorMap mapB1, const __grid_constant__ CUtensorMap mapB2) {
    extern __shared__ unsigned char smem_raw[];
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
    // everything above overlaps the previous kernel's tail; global memory is touched only below
    pdl_wait();
    pdl_launch_dependents();

    const TcPlan& p = a.p;
    const int it0 = blockIdx.x * p.U;
    const int it1 = min(it0 + p.U, p.tiles * p.KB);

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer ----------------
        const CUtensorMap* maps[3] = {&mapB0, &mapB1, &mapB2};
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int it = it0; it < it1 && ok;) {
            const int t = it / p.KB, kb0 = it - t * p.KB;
            const int kb1 = min(p.KB, kb0 + (it1 - it));
            const int mt = t / p.n_tiles, nt = t - mt * p.n_tiles;
            int row0, row1;
            const int s0 = half_source(a, nt, 0, row0), s1 = half_source(a, nt, 1, row1);
            const uint32_t bytes = TC_A_BYTES + TC_HALF_BYTES * (1 + (s1 >= 0));
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1, abort_flag))) break;
                const uint32_t sA = base + stage * TC_STAGE_BYTES, sB = sA + TC_A_BYTES;
                mbar_expect_tx(full_bar(stage), bytes);
                tma_load_2d(sA, &mapA, kb * TC_BK, mt * TC_BM, full_bar(stage));
                tma_load_2d(sB, maps[s0], kb * TC_BK, row0, full_bar(stage));
                if (s1 >= 0) tma_load_2d(sB + TC_HALF_BYTES, maps[s1], kb * TC_BK, row1, full_bar(stage));
                if (++stage == TC_STAGES) { stage = 0; phase ^= 1; }
            }
            it += kb1 - kb0;
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer ----------------
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ok = true;
        for (int it = it0; it < it1 && ok;) {
            const int t = it / p.KB, kb0 = it - t * p.KB;
            const int kb1 = min(p.KB, kb0 + (it1 - it));
            const int nt = t % p.n_tiles;
            int row1;
            const uint32_t idesc = idesc_bf16(half_source(a, nt, 1, row1) >= 0 ? 256 : 128);
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
    } else if (warp >= 2) {
        // ---------------- drain: TMEM -> fp32 partial tile ----------------
        const int q = warp & 3;                   // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int it = it0; it < it1 && ok;) {
            const int t = it / p.KB, kb0 = it - t * p.KB;
            const int kb1 = min(p.KB, kb0 + (it1 - it));
            const int mt = t / p.n_tiles, nt = t - mt * p.n_tiles;
            int row1;
            const int nchunks = half_source(a, nt, 1, row1) >= 0 ? 8 : 4;
            const int slot = blockIdx.x - (int)(((int64_t)t * p.KB) / p.U);
            float4* dst = reinterpret_cast<float4*>(a.partial + ((int64_t)t * p.smax + slot) * TC_SLOT_FLOATS);
            if (!(ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag))) break;
            tc_fence_after();
            const bool valid = mt * TC_BM + row < a.M;
            for (int c = 0; c < nchunks; ++c) {
                float v[32];
                tc_ld32(tmem_base + acc * TC_BN + c * 32 + ((uint32_t)(q * 32) << 16), v);
                if (valid) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dst[(c * 8 + i) * TC_BM + row] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            it += kb1 - kb0;
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

// ---- finish: ordered sum of the partial tiles + epilogue --------------------------------------
// One thread owns 4 adjacent output columns of one row (plus the 4 columns its epilogue pairs
// them with: the other rotary half, or the up-projection of a gate column).  A warp covers 32
// consecutive rows of the same columns, so every partial-tile read is one contiguous 512-byte
// segment; the slots are summed in ascending CTA order, which makes the result bitwise
// reproducible.
constexpr int FIN_ITEMS_PER_SUB = 2;   // items each half-block of 128 threads walks through

__device__ __forceinline__ float4 sum_slots(const float4* __restrict__ src, int nslots, int pc, int row) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4* q = src + pc * TC_BM + row;
#pragma unroll 4
    for (int c = 0; c < nslots; ++c) {
        const float4 v = __ldcg(q + (int64_t)c * (TC_SLOT_FLOATS / 4));
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    return s;
}

__device__ __forceinline__ uint2 pack4(float a, float b, float c, float d) {
    return make_uint2(pack_bf16(a, b), pack_bf16(c, d));
}

__global__ void __launch_bounds__(256) gemm_finish_kernel(const GemmArgs g, const TcPlan p, const float* __restrict__ partial,
                                                          int n_items) {
    pdl_wait();
    pdl_launch_dependents();
    const int row = threadIdx.x & 127, sub = threadIdx.x >> 7;
    const int mt = blockIdx.y, grow = mt * TC_BM + row;
    if (grow >= g.M) return;
    for (int k = 0; k < FIN_ITEMS_PER_SUB; ++k) {
        const int item = (blockIdx.x * 2 + sub) * FIN_ITEMS_PER_SUB + k;
        if (item >= n_items) return;
        int nt, pc0, pc1;            // N tile, partial column groups of the two halves
        int u128 = 0, r = 0;
        if (g.epilogue == kEpiResidual) {
            nt = item >> 6; pc0 = item & 63; pc1 = -1;
        } else if (g.epilogue == kEpiSwiGLU) {
            nt = item >> 5; pc0 = item & 31; pc1 = 32 + pc0;
        } else {
            u128 = item >> 4; r = item & 15;
            nt = u128 >> 1;
            const int c4 = g.head_dim == 128 ? r : ((r >> 3) << 4) + (r & 7);
            pc0 = 32 * (u128 & 1) + c4;
            pc1 = pc0 + (g.head_dim >> 3);
        }
        const int t = mt * p.n_tiles + nt;
        const int c_first = (int)(((int64_t)t * p.KB) / p.U);
        const int c_last = (int)(((int64_t)(t + 1) * p.KB - 1) / p.U);
        const int nslots = c_last - c_first + 1;
        const float4* src = reinterpret_cast<const float4*>(partial + (int64_t)t * p.smax * TC_SLOT_FLOATS);
        const float4 v0 = sum_slots(src, nslots, pc0, row);
        if (g.epilogue == kEpiResidual) {
            const int N = g.n[0], col = item * 4;
            const int64_t roff = g.resid_off ? g.resid_off[grow] : (int64_t)grow * N;
            const uint2 rv = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(g.resid) + roff + col);
            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(g.c) + (int64_t)grow * N + col) =
                pack4(v0.x + bf16_lo(rv.x), v0.y + bf16_hi(rv.x), v0.z + bf16_lo(rv.y), v0.w + bf16_hi(rv.y));
            continue;
        }
        const float4 v1 = sum_slots(src, nslots, pc1, row);
        if (g.epilogue == kEpiSwiGLU) {
            const float gt[4] = {v0.x, v0.y, v0.z, v0.w}, up[4] = {v1.x, v1.y, v1.z, v1.w};
            float o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) o[i] = gt[i] / (1.f + __expf(-gt[i])) * up[i];
            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(g.c) + (int64_t)grow * g.n[0] + item * 4) =
                pack4(o[0], o[1], o[2], o[3]);
            continue;
        }
        // q/k/v: bias, rotary embedding with the pairing (i, i + d/2), store (+ fused cache scatter)
        int seg = 0, c0 = u128 * 128;
        while (seg < 2 && c0 >= g.n[seg]) { c0 -= g.n[seg]; ++seg; }
        const int half = g.head_dim >> 1;
        const int j4 = (g.head_dim == 128 ? r : (r & 7)) * 4;               // index inside the half head
        const int col = c0 + (g.head_dim == 128 ? r * 4 : ((r >> 3) << 6) + (r & 7) * 4);
        float lo[4] = {v0.x, v0.y, v0.z, v0.w}, hi[4] = {v1.x, v1.y, v1.z, v1.w};
        const __nv_bfloat16* bias = static_cast<const __nv_bfloat16*>(g.bias[seg]);
        if (bias) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                lo[i] += __bfloat162float(bias[col + i]);
                hi[i] += __bfloat162float(bias[col + half + i]);
            }
        }
        const int pos = g.row_pos[grow];
        if (seg < g.rope_segments) {
            const int pp = pos < 0 ? 0 : pos;
            const float4 cs = *reinterpret_cast<const float4*>(g.rope_cos + (int64_t)pp * half + j4);
            const float4 sn = *reinterpret_cast<const float4*>(g.rope_sin + (int64_t)pp * half + j4);
            const float c[4] = {cs.x, cs.y, cs.z, cs.w}, sv[4] = {sn.x, sn.y, sn.z, sn.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float x = lo[i], y = hi[i];
                lo[i] = x * c[i] - y * sv[i];
                hi[i] = y * c[i] + x * sv[i];
            }
        }
        const uint2 plo = pack4(lo[0], lo[1], lo[2], lo[3]), phi = pack4(hi[0], hi[1], hi[2], hi[3]);
        const int nseg = g.n[seg];
        if (g.out[seg]) {
            __nv_bfloat16* o = static_cast<__nv_bfloat16*>(g.out[seg]) + (int64_t)grow * nseg + col;
            *reinterpret_cast<uint2*>(o) = plo;
            *reinterpret_cast<uint2*>(o + half) = phi;
        }
        __nv_bfloat16* cache = seg == 1 ? static_cast<__nv_bfloat16*>(g.cache_k)
                             : seg == 2 ? static_cast<__nv_bfloat16*>(g.cache_v) : nullptr;
        if (cache && pos >= 0) {
            const int b = grow / g.rows_per_req;
            __nv_bfloat16* o = cache + (int64_t)b * g.kv_batch_stride + (int64_t)pos * nseg + col;
            *reinterpret_cast<uint2*>(o) = plo;
            *reinterpret_cast<uint2*>(o + half) = phi;
        }
    }
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
constexpr int kMapCache = 64;
std::mutex g_map_mutex;
MapEntry g_maps[kMapCache];
int g_map_count = 0, g_map_next = 0;

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
    p.smax = (p.KB + p.U - 1) / p.U + 1;
    return p;
}

}  // namespace

size_t gemm_partial_bytes(int M, int K, int n_total, bool swiglu) {
    if (M <= 0) return 0;
    TcPlan p = make_plan(M, K, swiglu ? n_total / 128 : n_total / 128, swiglu);
    return (size_t)p.tiles * p.smax * TC_SLOT_FLOATS * sizeof(float);
}

int launch_gemm(const GemmArgs& g, cudaStream_t stream) {
    if (g.M == 0) return 0;
    static const bool use_mma = [] { const char* e = getenv("ACACHE_GEMM_IMPL"); return e && !strcmp(e, "mma"); }();
    if (use_mma) return launch_gemm_mma(g, stream);
    std::lock_guard<std::mutex> lock(g_map_mutex);
    const bool swiglu = g.epilogue == kEpiSwiGLU;
    const int n_total = swiglu ? g.n[0] : g.n[0] + g.n[1] + g.n[2];
    TcArgs a{};
    a.M = g.M;
    a.swiglu = swiglu;
    a.n[0] = g.n[0]; a.n[1] = g.n[1]; a.n[2] = g.n[2];
    a.p = make_plan(g.M, g.K, n_total / 128, swiglu);
    a.partial = g.partial;
    a.status = g.status;
    const CUtensorMap* mA = get_map(g.a, g.M, g.K);
    const CUtensorMap* mB[3] = {nullptr, nullptr, nullptr};
    for (int i = 0; i < 3; ++i)
        if (g.b[i]) mB[i] = get_map(g.b[i], swiglu ? g.n[0] : g.n[i], g.K);
    if (!mA || !mB[0]) return -1;
    for (int i = 1; i < 3; ++i)
        if (!mB[i]) mB[i] = mB[0];
    static bool attr = false;
    if (!attr) {
        cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM);
        attr = true;
    }
    launch_pdl(gemm_tc_kernel, a.p.ctas, TC_THREADS, TC_SMEM, stream, a, *mA, *mB[0], *mB[1], *mB[2]);
    const int n_items = g.epilogue == kEpiQKV ? n_total / 8 : n_total / 4;
    const int per_cta = 2 * FIN_ITEMS_PER_SUB;
    launch_pdl(gemm_finish_kernel, dim3((n_items + per_cta - 1) / per_cta, a.p.m_tiles), 256, 0, stream, g, a.p,
               (const float*)g.partial, n_items);
    return 2;
}

}  // namespace acache
