// Query absorption Q_A = Q_N W_UK (Algorithm 1 line 5) on tcgen05 / TMEM / TMA.
//
// Per head h: Q_A[b, h, :] = q_nope[b, h, :] (1 x 128) * W_UK[h] (128 x 512).  A CTA owns one
// head and up to 128 requests.  Both operands fit shared memory at once (q tile 32 KB, the
// head's transposed weight 128 KB), so all TMA loads are issued up front and the 512-wide
// result is accumulated in all 512 tensor-memory columns (four N = 128 tiles).  The step is
// bound by reading the 16.8 MB of weights once; its cost is one load latency plus the stream.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2-5 = epilogue (tcgen05.ld, bf16 pack, store).
#include "kernels.h"
#include "sm100.cuh"



namespace tmla {
namespace {

using namespace sm100;

constexpr int A_BYTES = 128 * 128 * 2;        // 2 slabs [128 rows][64]
constexpr int W_BYTES = 512 * 128 * 2;        // 4 N-tiles x 2 slabs [128 rows][64]
constexpr int SMEM_BYTES = A_BYTES + W_BYTES + 1024 + 256;

struct QAbsorbParams {
    void* q_abs;   // bf16 [B, H, 512]
    int B, H;
    int* status;
    // optional: one extra block (blockIdx.y == H) computes the longest-first request order that the
    // absorb attention kernel launched next uses, saving a launch on the absorb branch
    const int32_t* seq_lens;
    int32_t* order;
    // optional per-position descriptors for the absorb kernel
    const int32_t* block_table;
    int max_pages, page_size;
    int4* desc;
};

__global__ void __launch_bounds__(192, 1)
q_absorb_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_w, QAbsorbParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    pdl_trigger();
    pdl_wait();
    if ((int)blockIdx.y == p.H) {   // the ordering block (whole block takes this branch)
        if (blockIdx.x == 0) {
            block_order_by_length(p.seq_lens, p.B, p.order, reinterpret_cast<unsigned long long*>(smem));
            if (p.desc != nullptr) {
                __syncthreads();   // perm[] written by this block is read back below
                for (int i = threadIdx.x; i < p.B; i += blockDim.x) {
                    const int b = p.order[i];
                    const int len = min(max(p.seq_lens[b], 0), p.max_pages * p.page_size);
                    const int32_t* bt = p.block_table + (int64_t)b * p.max_pages;
                    p.desc[i] = make_int4(b, len, p.max_pages > 0 ? bt[0] : -1, p.max_pages > 1 ? bt[1] : -1);
                }
            }
        }
        return;
    }
    uint8_t* sA = smem;
    uint8_t* sW = smem + A_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(sW + W_BYTES);   // [0..3]: q + weight tile n ; [4]: accumulators done
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(full + 5);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    const int b0 = blockIdx.x * 128, h = blockIdx.y;

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < 5; ++i) mbar_init(&full[i], 1);
            *abort_flag = 0;
            fence_mbar_init();
        }
        __syncwarp();
        const uint32_t ld = elect_one() ? 1u : 0u;
        // barrier n completes when weight tile n (and, for n = 0, the q tile) has landed
        mbar_arrive_expect_tx_if(ld, &full[0], A_BYTES + W_BYTES / 4);
        tma_load_3d_if(ld, sA, &tm_q, &full[0], 0, h, b0);
        tma_load_3d_if(ld, sA + 16384, &tm_q, &full[0], 64, h, b0);
#pragma unroll 1
        for (int n = 0; n < 4; ++n) {
            if (n > 0) mbar_arrive_expect_tx_if(ld, &full[n], W_BYTES / 4);
            tma_load_3d_if(ld, sW + n * 32768, &tm_w, &full[n], 0, n * 128, h);
            tma_load_3d_if(ld, sW + n * 32768 + 16384, &tm_w, &full[n], 64, n * 128, h);
        }
    }
    if (warp == 1) tmem_alloc(tmem_holder, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_holder, 0);

    if (warp == 1) {
        const uint32_t ld = elect_one() ? 1u : 0u;
        constexpr uint32_t idesc = idesc_bf16(128, 128, false, false);
        bool ok = true;
        for (int n = 0; n < 4 && ok; ++n) {
            ok = mbar_wait_warp(&full[n], 0, abort_flag);
            if (!ok) break;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                const uint64_t da = smem_desc_k_sw128(smem_u32(sA + ks * 16384));
                const uint64_t db = smem_desc_k_sw128(smem_u32(sW + n * 32768 + ks * 16384));
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_ss_if(ld, tmem_base + n * 128, da + 2 * k, db + 2 * k, idesc, (ks | k) != 0);
            }
        }
        if (ok) umma_commit_if(ld, &full[4]);
    } else if (warp >= 2) {
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&full[4], 0, abort_flag));
        tc_fence_after();
        if (ok) {
            const int lg = (warp & 3) * 32;
            const int b = b0 + lg + lane;
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.q_abs) + ((int64_t)b * p.H + h) * 512;
#pragma unroll 1
            for (int c = 0; c < 16; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)lg << 16) + c * 32, r);
                tmem_ld_wait();
                if (b < p.B) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(r[j * 8 + 0]), __uint_as_float(r[j * 8 + 1]));
                        v.y = pack_bf16(__uint_as_float(r[j * 8 + 2]), __uint_as_float(r[j * 8 + 3]));
                        v.z = pack_bf16(__uint_as_float(r[j * 8 + 4]), __uint_as_float(r[j * 8 + 5]));
                        v.w = pack_bf16(__uint_as_float(r[j * 8 + 6]), __uint_as_float(r[j * 8 + 7]));
                        *reinterpret_cast<uint4*>(dst + c * 32 + j * 8) = v;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // A wait gave up: all copies of this CTA were issued up front against full[0..3]; wait for them (with a limit)
        // before the shared memory is released, then report.
        if (warp == 0)
            for (int n = 0; n < 4; ++n) mbar_drain(&full[n], 0);
        if (threadIdx.x == 0 && p.status) atomicOr(p.status, 4);
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace

cudaError_t set_attrs_q_absorb_sm100() {
    return cudaFuncSetAttribute(q_absorb_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}

cudaError_t make_q_absorb_tmap(const void* w_uk_t, int H, CUtensorMap* tm_w) {
    uint64_t dims[3] = {128, 512, (uint64_t)H};
    uint64_t str[2] = {128 * 2, 512 * 128 * 2};
    uint32_t box[3] = {64, 128, 1};
    return make_tmap_bf16(tm_w, w_uk_t, 3, dims, str, box);
}

cudaError_t launch_q_absorb_sm100(const void* q_nope, const CUtensorMap* tm_w, void* q_abs, int B, int H, int* status,
                                  const int32_t* seq_lens, int32_t* order, const int32_t* block_table, int max_pages,
                                  int page_size, int32_t* desc, cudaStream_t s) {
    if (B <= 0) return cudaSuccess;
    CUtensorMap tm_q;
    uint64_t dims[3] = {128, (uint64_t)H, (uint64_t)B};
    uint64_t str[2] = {128 * 2, (uint64_t)H * 128 * 2};
    uint32_t box[3] = {64, 1, 128};
    cudaError_t e = make_tmap_bf16(&tm_q, q_nope, 3, dims, str, box);
    if (e != cudaSuccess) return e;
    const bool with_order = seq_lens != nullptr && order != nullptr && B <= 4096;
    QAbsorbParams p{q_abs, B, H, status, seq_lens, order, block_table, max_pages, page_size,
                    (with_order && block_table != nullptr) ? reinterpret_cast<int4*>(desc) : nullptr};
    dim3 grid((B + 127) / 128, H + (with_order ? 1 : 0), 1);
    return launch_pdl(q_absorb_sm100_kernel, grid, dim3(192), SMEM_BYTES, s, tm_q, *tm_w, p);
}

}  // namespace tmla
