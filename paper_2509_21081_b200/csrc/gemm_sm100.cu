// Batched bf16 GEMM on the 5th-generation tensor cores:
//   C[z][m][n] = sum_k A[z][m][k] * B[z][n][k]      (both operands K-major)
// TMA stages 128 x 64 operand tiles (128-byte swizzle) into shared memory, one
// elected thread issues tcgen05.mma into a 128 x 128 fp32 accumulator in tensor
// memory, four warps read it back with tcgen05.ld and store bf16.
// Used for the shared-prefix expansion (Section 3.1 "Prefill"), where it is a
// large dense contraction: [L_s, 512] x [512, 128] per head for K and V.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 2-5 = epilogue (one 32-lane TMEM slice each).
#include "kernels.h"
#include "sm100.cuh"



namespace tmla {
namespace {

using namespace sm100;

constexpr int BM = 128, BN = 128, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

struct GemmParams {
    void* C; int64_t ldc, c_batch;
    int M, N, K, c_block_n, c_tile64;
    int a_batched, b_batched, a_swap;
    int* status;
    int out_mode;          // 0: bf16 C, 1: fp32 C, 2: LSE combine epilogue (N == 128, row = request, batch = head)
    CombineEpilogue ce;
};

__global__ void __launch_bounds__(192) gemm_tn_sm100_kernel(const __grid_constant__ CUtensorMap tmA,
                                                            const __grid_constant__ CUtensorMap tmB, GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_full + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * BM, z = blockIdx.z;
    pdl_trigger();
    pdl_wait();
    const int KB = p.K / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init(acc_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) tmem_alloc(tmem_holder, 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_holder, 0);

    int kb_issued = 0;   // producer warp: operand tiles issued (upper bound), for the abort path
    if (warp == 0) {
        // producer: the whole warp runs the loop, the elected lane issues
        const uint32_t ld = elect_one() ? 1u : 0u;
        for (int kb = 0; kb < KB; ++kb) {
            const int s = kb % STAGES;
            if (!mbar_wait_warp(&empty[s], ((kb / STAGES) & 1) ^ 1, abort_flag)) break;
            kb_issued = kb + 1;
            mbar_arrive_expect_tx_if(ld, &full[s], STAGE_BYTES);
            uint8_t* sa = smem + s * STAGE_BYTES;
            if (p.a_swap) tma_load_3d_if(ld, sa, &tmA, &full[s], kb * BK, z, m0);
            else tma_load_3d_if(ld, sa, &tmA, &full[s], kb * BK, m0, p.a_batched ? z : 0);
            tma_load_3d_if(ld, sa + A_BYTES, &tmB, &full[s], kb * BK, n0, p.b_batched ? z : 0);
        }
    } else if (warp == 1) {
        const uint32_t ld = elect_one() ? 1u : 0u;
        constexpr uint32_t idesc = idesc_bf16(BM, BN, false, false);
        bool ok = true;
        for (int kb = 0; kb < KB && ok; ++kb) {
            const int s = kb % STAGES;
            ok = mbar_wait_warp(&full[s], (kb / STAGES) & 1, abort_flag);
            if (!ok) break;
            const uint32_t sa = smem_u32(smem + s * STAGE_BYTES);
            const uint64_t da = smem_desc_k_sw128(sa), db = smem_desc_k_sw128(sa + A_BYTES);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k) umma_ss_if(ld, tmem_base, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
            umma_commit_if(ld, &empty[s]);
        }
        if (ok) umma_commit_if(ld, acc_full);
    } else {
        const int lg = (warp & 3) * 32;
        const int row = m0 + lg + lane;
        // Combine epilogue, first half: while the main loop runs, this thread (one request row) reads the
        // LSEs of its (request, head), derives the merge weights and accumulates the weighted naive-side
        // partials in registers, so that their memory latency is hidden behind the GEMM.
        float accn[128];
        float wa = 0.f, inv = 0.f, m = -INFINITY, zsum = 0.f;
        int64_t bh = 0;
        const bool live = p.out_mode == 2 && row < p.M;
        if (p.out_mode == 2) {
            const CombineEpilogue& ce = p.ce;
            const int64_t BH = (int64_t)p.M * ce.H;
            bh = (int64_t)row * ce.H + z;
#pragma unroll
            for (int q = 0; q < 128; ++q) accn[q] = 0.f;
            if (live) {
                const float la = ce.lse_abs[bh];
                m = la;
                for (int i = 0; i < ce.n_naive; ++i) m = fmaxf(m, ce.lse_naive[i * BH + bh]);
                if (m != -INFINITY) {
                    wa = (la == -INFINITY) ? 0.f : __expf(la - m);
                    zsum = wa;
                    for (int i = 0; i < ce.n_naive; ++i) {
                        const float l = ce.lse_naive[i * BH + bh];
                        if (l == -INFINITY) continue;          // empty partial: its O slot was never written
                        const float w = __expf(l - m);
                        zsum += w;
                        const float4* src = reinterpret_cast<const float4*>(ce.o_naive + (i * BH + bh) * 128);
#pragma unroll
                        for (int q = 0; q < 32; ++q) {
                            const float4 v = src[q];
                            accn[4 * q] += w * v.x; accn[4 * q + 1] += w * v.y; accn[4 * q + 2] += w * v.z; accn[4 * q + 3] += w * v.w;
                        }
                    }
                }
                inv = zsum > 0.f ? 1.f / zsum : 0.f;
            }
        }
        const bool ok = __all_sync(0xffffffffu, mbar_wait(acc_full, 0, abort_flag));
        tc_fence_after();
        if (ok) {
            if (p.out_mode == 2) {
                // second half: add the absorb-side row (the accumulator, already normalised) with its weight,
                // normalise (Algorithm 1 line 8) and write the final bf16 row
                const CombineEpilogue& ce = p.ce;
#pragma unroll
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)lg << 16) + c * 32, r);
                    tmem_ld_wait();
                    if (!live) continue;
                    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(ce.out) + bh * 128 + c * 32;
                    float* dstf = reinterpret_cast<float*>(ce.out) + bh * 128 + c * 32;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float o[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float oa = wa > 0.f ? wa * __uint_as_float(r[j * 8 + e]) : 0.f;
                            o[e] = (accn[c * 32 + j * 8 + e] + oa) * inv;
                        }
                        if (ce.out_fp32) {
                            *reinterpret_cast<float4*>(dstf + j * 8) = make_float4(o[0], o[1], o[2], o[3]);
                            *reinterpret_cast<float4*>(dstf + j * 8 + 4) = make_float4(o[4], o[5], o[6], o[7]);
                        } else {
                            uint4 v;
                            v.x = pack_bf16(o[0], o[1]); v.y = pack_bf16(o[2], o[3]);
                            v.z = pack_bf16(o[4], o[5]); v.w = pack_bf16(o[6], o[7]);
                            *reinterpret_cast<uint4*>(dst + j * 8) = v;
                        }
                    }
                }
                if (live && ce.lse_out) ce.lse_out[bh] = (m == -INFINITY) ? -INFINITY : m + __logf(zsum);
            } else {
                uint8_t* cbase = reinterpret_cast<uint8_t*>(p.C) + (int64_t)z * p.c_batch * (p.out_mode == 1 ? 4 : 2);
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)lg << 16) + c * 32, r);
                    tmem_ld_wait();
                    if (row < p.M) {
                        const int gn = n0 + c * 32;
                        const int64_t off = p.c_tile64 ? (((int64_t)(row >> 6) * (p.N >> 6) + (gn >> 6)) << 12) + ((row & 63) << 6) + (gn & 63)
                                            : p.c_block_n ? ((int64_t)(gn >> 6) * p.M + row) * 64 + (gn & 63)
                                                          : (int64_t)row * p.ldc + gn;
                        if (p.out_mode == 1) {
                            float4* crow = reinterpret_cast<float4*>(cbase + off * 4);
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                crow[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                      __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                        } else {
                            __nv_bfloat16* crow = reinterpret_cast<__nv_bfloat16*>(cbase + off * 2);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                uint4 v;
                                v.x = pack_bf16(__uint_as_float(r[j * 8 + 0]), __uint_as_float(r[j * 8 + 1]));
                                v.y = pack_bf16(__uint_as_float(r[j * 8 + 2]), __uint_as_float(r[j * 8 + 3]));
                                v.z = pack_bf16(__uint_as_float(r[j * 8 + 4]), __uint_as_float(r[j * 8 + 5]));
                                v.w = pack_bf16(__uint_as_float(r[j * 8 + 6]), __uint_as_float(r[j * 8 + 7]));
                                *reinterpret_cast<uint4*>(crow + j * 8) = v;
                            }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // A wait gave up: before the CTA's shared memory is released the producer warp waits (with a limit) for the
        // operand tiles it issued last, the only copies that can still be in flight; then report.
        if (warp == 0)
            for (int kb = max(0, kb_issued - STAGES); kb < kb_issued; ++kb) mbar_drain(&full[kb % STAGES], (kb / STAGES) & 1);
        if (threadIdx.x == 0 && p.status) atomicOr(p.status, 1);
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem_base, 128);
}

}  // namespace

cudaError_t set_attrs_gemm_sm100() {
    return cudaFuncSetAttribute(gemm_tn_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}

cudaError_t launch_gemm_tn_sm100(const GemmTN& g, int* status, cudaStream_t s, const CombineEpilogue* ce) {
    if (g.M <= 0 || g.batch <= 0) return cudaSuccess;
    if (g.N % BN != 0 || g.K % BK != 0) return cudaErrorInvalidValue;
    if (ce && g.N != BN) return cudaErrorInvalidValue;
    CUtensorMap tmA, tmB;
    // When the batch stride of A is smaller than its row stride (activations laid out [M, batch, K]) the
    // tensor map is built with the batch dimension in the middle so that strides stay increasing.
    const bool a_swap = g.a_batch != 0 && g.a_batch < g.lda;
    if (a_swap) {
        uint64_t dims[3] = {(uint64_t)g.K, (uint64_t)g.batch, (uint64_t)g.M};
        uint64_t strides[2] = {(uint64_t)g.a_batch * 2, (uint64_t)g.lda * 2};
        uint32_t box[3] = {BK, 1, BM};
        cudaError_t e = make_tmap_bf16(&tmA, g.A, 3, dims, strides, box);
        if (e != cudaSuccess) return e;
    } else {
        const bool batched = g.a_batch != 0;
        uint64_t dims[3] = {(uint64_t)g.K, (uint64_t)g.M, (uint64_t)(batched ? g.batch : 1)};
        uint64_t strides[2] = {(uint64_t)g.lda * 2, (uint64_t)(batched ? g.a_batch : (int64_t)g.lda * g.M) * 2};
        uint32_t box[3] = {BK, BM, 1};
        cudaError_t e = make_tmap_bf16(&tmA, g.A, 3, dims, strides, box);
        if (e != cudaSuccess) return e;
    }
    {
        const bool batched = g.b_batch != 0;
        uint64_t dims[3] = {(uint64_t)g.K, (uint64_t)g.N, (uint64_t)(batched ? g.batch : 1)};
        uint64_t strides[2] = {(uint64_t)g.ldb * 2, (uint64_t)(batched ? g.b_batch : (int64_t)g.ldb * g.N) * 2};
        uint32_t box[3] = {BK, BN, 1};
        cudaError_t e = make_tmap_bf16(&tmB, g.B, 3, dims, strides, box);
        if (e != cudaSuccess) return e;
    }
    GemmParams p{g.C, g.ldc, g.c_batch, g.M, g.N, g.K, g.c_block_n, g.c_tile64 ? 1 : 0, g.a_batch != 0, g.b_batch != 0, a_swap ? 1 : 0, status,
                 ce ? 2 : (g.out_fp32 ? 1 : 0), ce ? *ce : CombineEpilogue{}};
    dim3 grid(g.N / BN, (g.M + BM - 1) / BM, g.batch);
    return launch_pdl(gemm_tn_sm100_kernel, grid, dim3(192), SMEM_BYTES, s, tmA, tmB, p);
}

}  // namespace tmla
