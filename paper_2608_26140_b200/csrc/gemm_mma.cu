// C[M, N] = A[M, K] * B[N, K]^T in bf16 with fp32 accumulation, for the projections of the
// selective recomputation (Section 3.3): q/k/v of the recomputed rows, the attention output
// projection and the SwiGLU MLP.  This main loop uses warp-level mma.sync tiles fed by a
// cp.async pipeline; the epilogues are in gemm_epilogue.cuh.
#include "common.cuh"
#include "gemm_epilogue.cuh"
#include "kernels.h"

namespace acache {

constexpr int BM = 128, BN = 128, BK = 64, STAGES = 3, GEMM_THREADS = 256;
constexpr int A_TILE = BM * BK * 2, B_TILE = BN * BK * 2, STAGE_BYTES = A_TILE + B_TILE;
constexpr int GEMM_SMEM = STAGES * STAGE_BYTES;   // 96 KB, also covers the 66 KB epilogue staging
static_assert(GEMM_SMEM >= 128 * kStagePitch * 4, "staging must fit in the pipeline buffers");

// The weight row that tile row `r` (0..127) of N-tile `nt` reads, as a pointer to its start.
__device__ __forceinline__ const __nv_bfloat16* b_row_ptr(const GemmArgs& g, int seg, int seg_row0, int r, int nt) {
    if (g.epilogue == kEpiSwiGLU) {
        const __nv_bfloat16* w = static_cast<const __nv_bfloat16*>(g.b[r >> 6]);
        return w + (int64_t)(nt * 64 + (r & 63)) * g.K;
    }
    return static_cast<const __nv_bfloat16*>(g.b[seg]) + (int64_t)(seg_row0 + r) * g.K;
}

__global__ void __launch_bounds__(GEMM_THREADS) gemm_mma_kernel(const GemmArgs g) {
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp >> 2, wn = warp & 3;      // 2 x 4 warps, warp tile 64 x 32
    const int nt = blockIdx.x, m0 = blockIdx.y * BM;

    // which B segment this N tile falls in
    int seg = 0, seg_row0 = nt * BN;
    if (g.epilogue != kEpiSwiGLU) {
        while (seg < 2 && seg_row0 >= g.n[seg]) { seg_row0 -= g.n[seg]; ++seg; }
    }
    const __nv_bfloat16* A = static_cast<const __nv_bfloat16*>(g.a);
    const int KT = g.K / BK;

    auto load_stage = [&](int kt, int buf) {
        const uint32_t sa = sbase + buf * STAGE_BYTES, sb = sa + A_TILE;
        const int k0 = kt * BK;
#pragma unroll
        for (int i = 0; i < (BM * 8) / GEMM_THREADS; ++i) {
            int c = tid + i * GEMM_THREADS;
            int r = c >> 3, cc = c & 7;
            int ok = (m0 + r) < g.M;
            cp_async16(sa + swz64(r, cc), A + (int64_t)(ok ? m0 + r : 0) * g.K + k0 + cc * 8, ok ? 16 : 0);
        }
#pragma unroll
        for (int i = 0; i < (BN * 8) / GEMM_THREADS; ++i) {
            int c = tid + i * GEMM_THREADS;
            int r = c >> 3, cc = c & 7;
            cp_async16(sb + swz64(r, cc), b_row_ptr(g, seg, seg_row0, r, nt) + k0 + cc * 8, 16);
        }
    };

    float acc[4][4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[i][j][k] = 0.f;

    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < KT) load_stage(s, s);
        cp_async_commit();
    }
    for (int kt = 0; kt < KT; ++kt) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        if (kt + STAGES - 1 < KT) load_stage(kt + STAGES - 1, (kt + STAGES - 1) % STAGES);
        cp_async_commit();
        const uint32_t sa = sbase + (kt % STAGES) * STAGE_BYTES, sb = sa + A_TILE;
#pragma unroll
        for (int ks = 0; ks < BK / 16; ++ks) {
            uint32_t af[4][4], bf[4][2];
#pragma unroll
            for (int mi = 0; mi < 4; ++mi) {
                int r = wm * 64 + mi * 16 + (lane & 15);
                ldmatrix_x4(af[mi][0], af[mi][1], af[mi][2], af[mi][3], sa + swz64(r, ks * 2 + (lane >> 4)));
            }
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                int n = wn * 32 + np * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldmatrix_x4(bf[np * 2][0], bf[np * 2][1], bf[np * 2 + 1][0], bf[np * 2 + 1][1],
                            sb + swz64(n, ks * 2 + ((lane >> 3) & 1)));
            }
#pragma unroll
            for (int mi = 0; mi < 4; ++mi)
#pragma unroll
                for (int ni = 0; ni < 4; ++ni) mma_bf16_16816(acc[mi][ni], af[mi], bf[ni][0], bf[ni][1]);
        }
    }
    cp_async_wait<0>();
    __syncthreads();

    // stage the accumulators, then run the epilogue over whole rows
    float* stage = reinterpret_cast<float*>(smem);
#pragma unroll
    for (int mi = 0; mi < 4; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) {
            int r = wm * 64 + mi * 16 + (lane >> 2);
            int c = wn * 32 + ni * 8 + (lane & 3) * 2;
            *reinterpret_cast<float2*>(stage + r * kStagePitch + c) = make_float2(acc[mi][ni][0], acc[mi][ni][1]);
            *reinterpret_cast<float2*>(stage + (r + 8) * kStagePitch + c) = make_float2(acc[mi][ni][2], acc[mi][ni][3]);
        }
    __syncthreads();
    if (g.epilogue == kEpiQKV) epilogue_qkv(g, stage, m0, seg, seg_row0, tid, GEMM_THREADS);
    else if (g.epilogue == kEpiResidual) epilogue_residual(g, stage, m0, nt * BN, g.n[0], tid, GEMM_THREADS);
    else epilogue_swiglu(g, stage, m0, nt * 64, g.n[0], tid, GEMM_THREADS);
}

int launch_gemm_mma(const GemmArgs& g, cudaStream_t stream) {
    if (g.M == 0) return 0;
    int ntiles;
    if (g.epilogue == kEpiSwiGLU) ntiles = g.n[0] / 64;
    else ntiles = (g.n[0] + g.n[1] + g.n[2]) / BN;
    cudaFuncSetAttribute(gemm_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM);
    dim3 grid(ntiles, (g.M + BM - 1) / BM);
    gemm_mma_kernel<<<grid, GEMM_THREADS, GEMM_SMEM, stream>>>(g);
    return 1;
}

}  // namespace acache
