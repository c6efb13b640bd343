// Batched bf16 GEMM, both operands K-major:  C[z][m][n] = sum_k A[z][m][k] * B[z][n][k].
//
// Used for the three projection steps of the path: the shared-prefix expansion
// (Section 3.1 "Prefill"), the query absorption Q_A = Q_N W_KVb1 (Algorithm 1
// line 5) and the output projection O_A W_KVb2^T (Algorithm 1 line 7).  At
// decode time these are weight-read bound (16.8 MB per projection at H = 128),
// so warp-level tensor-core MMA with a cp.async pipeline is sufficient.
//
// Tile 128 x 128 x 32, 256 threads (2 x 4 warps, warp tile 64 x 32), 3 stages.
// Requirements: N % 128 == 0, K % 32 == 0, 16-byte aligned rows; M is ragged
// (rows >= M are zero-filled on load and skipped on store).
#include "common.cuh"
#include "kernels.h"

namespace tmla {
namespace {

constexpr int BM = 128, BN = 128, BK = 32, STAGES = 3;
constexpr int STAGE_ELEMS = (BM + BN) * BK;

// 64-byte rows, four 16-byte chunks per row; XOR swizzle keeps ldmatrix conflict-free.
__device__ __forceinline__ int sw_off(int row, int chunk) { return row * BK + ((chunk ^ ((row >> 1) & 3)) << 3); }

template <bool OUT_FP32>
__global__ void __launch_bounds__(256) gemm_tn_kernel(GemmTN g) {
    extern __shared__ __align__(128) __nv_bfloat16 smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp >> 2, wn = warp & 3;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * BM, z = blockIdx.z;
    const __nv_bfloat16* A = reinterpret_cast<const __nv_bfloat16*>(g.A) + (int64_t)z * g.a_batch;
    const __nv_bfloat16* B = reinterpret_cast<const __nv_bfloat16*>(g.B) + (int64_t)z * g.b_batch;

    auto load_stage = [&](int stage, int k0) {
        __nv_bfloat16* sA = smem + stage * STAGE_ELEMS;
        __nv_bfloat16* sB = sA + BM * BK;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            int idx = tid + i * 256;
            int row = idx >> 2, ch = idx & 3;
            int gm = m0 + row;
            bool ok = gm < g.M;
            const __nv_bfloat16* src = A + (int64_t)(ok ? gm : 0) * g.lda + k0 + ch * 8;
            cp_async16(smem_u32(sA + sw_off(row, ch)), src, ok);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            int idx = tid + i * 256;
            int row = idx >> 2, ch = idx & 3;
            const __nv_bfloat16* src = B + (int64_t)(n0 + row) * g.ldb + k0 + ch * 8;
            cp_async16(smem_u32(sB + sw_off(row, ch)), src, true);
        }
    };

    float acc[4][4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[i][j][k] = 0.f;

    const int KT = g.K / BK;
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < KT) load_stage(s, s * BK);
        cp_async_commit();
    }
    for (int kt = 0; kt < KT; ++kt) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        {
            int nk = kt + STAGES - 1;
            if (nk < KT) load_stage(nk % STAGES, nk * BK);
            cp_async_commit();
        }
        const __nv_bfloat16* sA = smem + (kt % STAGES) * STAGE_ELEMS;
        const __nv_bfloat16* sB = sA + BM * BK;
#pragma unroll
        for (int ks = 0; ks < BK / 16; ++ks) {
            uint32_t a[4][4], b[2][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int row = wm * 64 + i * 16 + (lane & 15);
                int ch = ks * 2 + (lane >> 4);
                ldmatrix_x4(a[i], smem_u32(sA + sw_off(row, ch)));
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                int row = wn * 32 + j * 16 + (lane & 7) + ((lane >> 4) << 3);
                int ch = ks * 2 + ((lane >> 3) & 1);
                ldmatrix_x4(b[j], smem_u32(sB + sw_off(row, ch)));
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) mma_bf16(acc[i][j], a[i], b[j >> 1][(j & 1) * 2], b[j >> 1][(j & 1) * 2 + 1]);
        }
    }
    cp_async_wait<0>();

    // epilogue
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            int gm = m0 + wm * 64 + i * 16 + (lane >> 2) + half * 8;
            if (gm >= g.M) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int gn = n0 + wn * 32 + j * 8 + (lane & 3) * 2;
                float v0 = acc[i][j][half * 2], v1 = acc[i][j][half * 2 + 1];
                const int64_t off = g.c_tile64 ? (((int64_t)(gm >> 6) * (g.N >> 6) + (gn >> 6)) << 12) + ((gm & 63) << 6) + (gn & 63)
                                    : g.c_block_n ? ((int64_t)(gn >> 6) * g.M + gm) * 64 + (gn & 63)
                                                  : (int64_t)gm * g.ldc + gn;
                if (OUT_FP32) {
                    float* C = reinterpret_cast<float*>(g.C) + (int64_t)z * g.c_batch + off;
                    *reinterpret_cast<float2*>(C) = make_float2(v0, v1);
                } else {
                    __nv_bfloat16* C = reinterpret_cast<__nv_bfloat16*>(g.C) + (int64_t)z * g.c_batch + off;
                    *reinterpret_cast<uint32_t*>(C) = pack_bf16(v0, v1);
                }
            }
        }
    }
}

}  // namespace

cudaError_t launch_gemm_tn(const GemmTN& g, cudaStream_t s) {
    if (g.M <= 0 || g.batch <= 0) return cudaSuccess;
    if (g.N % BN != 0 || g.K % BK != 0) return cudaErrorInvalidValue;
    dim3 grid(g.N / BN, (g.M + BM - 1) / BM, g.batch);
    size_t smem = (size_t)STAGES * STAGE_ELEMS * sizeof(__nv_bfloat16);
    if (g.out_fp32) gemm_tn_kernel<true><<<grid, 256, smem, s>>>(g);
    else gemm_tn_kernel<false><<<grid, 256, smem, s>>>(g);
    return cudaGetLastError();
}

cudaError_t set_attrs_gemm_tn() {
    const int smem = (int)((size_t)STAGES * STAGE_ELEMS * sizeof(__nv_bfloat16));
    cudaError_t e = cudaFuncSetAttribute(gemm_tn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return e;
}

}  // namespace tmla
