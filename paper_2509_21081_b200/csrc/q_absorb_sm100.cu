// Query absorption Q_A = Q_N W_UK (Algorithm 1 line 5) on tcgen05 / TMEM / TMA.
//
// Per head h: Q_A[b, h, :] = q_nope[b, h, :] (1 x 128) * W_UK[h] (128 x 512).  A CTA owns one head and every
// S-th tile of 128 requests (S CTAs per head when there are more SMs than heads).  The head's transposed weight
// (128 KB) is loaded once and stays in shared memory; the query tiles (32 KB) stream through one buffer that is
// refilled as soon as the products that read it have completed, i.e. while the previous tile's result is still
// being written.  With at most 128 requests (one tile per head) the grid may instead be a few CTAs that each walk
// through every G-th head ("walk" mode): in a hybrid step the kernel runs on the few SMs the shared-prefix kernel
// leaves free, and a CTA that stays resident loads the next head's weights while the previous head's result is
// being written, instead of paying launch, barrier set-up and tensor-memory allocation once per head.  The 512-wide result of a tile is accumulated in all 512 tensor-memory columns (four N = 128
// blocks).  The epilogue packs each block to bf16 into a 128-byte-swizzled staging buffer (two of them, used
// alternately) and writes it with tiled bulk stores, so that global memory sees whole 128-byte lines instead
// of one 16-byte piece per thread.  The step is bound by reading the weights once (16.8 MB at 128 heads) and
// by writing Q_A (1 KB per (request, head)).
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2-5 = epilogue (tcgen05.ld, bf16 pack, staged store).
#include <algorithm>

#include "kernels.h"
#include "sm100.cuh"

namespace tmla {
namespace {

using namespace sm100;

constexpr int A_BYTES = 128 * 128 * 2;        // 2 slabs [128 rows][64]
constexpr int W_BYTES = 512 * 128 * 2;        // 4 N-tiles x 2 slabs [128 rows][64]
constexpr int STAGE_BYTES = 128 * 128 * 2;    // one N = 128 block of the result: 2 slabs [128 rows][64]
constexpr int SMEM_BYTES = A_BYTES + W_BYTES + 2 * STAGE_BYTES + 1024 + 256;

struct QAbsorbParams {
    void* q_abs;   // bf16 [B, H, 512]
    int B, H;
    int n_tiles, splits;   // tiles of 128 requests; CTAs per head (CTA s takes tiles s, s + splits, ...)
    int walk_ctas;         // > 0: walk mode with this many working CTAs (1-D grid, block walk_ctas is the ordering block)
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
q_absorb_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_w,
                      const __grid_constant__ CUtensorMap tm_out, QAbsorbParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    pdl_trigger();
    pdl_wait();
    const bool walk = p.walk_ctas > 0;
    if (walk ? (int)blockIdx.x == p.walk_ctas : (int)blockIdx.y == p.H) {   // the ordering block (whole block takes this branch)
        if (walk || blockIdx.x == 0) {
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
    uint8_t* sOut = sW + W_BYTES;                                  // 2 staging buffers
    uint64_t* w_full = reinterpret_cast<uint64_t*>(sOut + 2 * STAGE_BYTES);   // [0..3]: weight block n has landed
    uint64_t* q_full = w_full + 4;      // query tile t has landed (phase t)
    uint64_t* acc_full = w_full + 5;    // the products of tile t are complete (phase t): accumulators ready, query buffer free
    uint64_t* acc_empty = w_full + 6;   // the epilogue has read the accumulators of tile t (128 arrivals, phase t)
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(w_full + 7);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    // work items of this CTA: (head, request tile).  Walk mode: heads blockIdx.x, + walk_ctas, ..., tile 0 each.
    const int n_my = walk ? (((int)blockIdx.x < p.H) ? (p.H - 1 - (int)blockIdx.x) / p.walk_ctas + 1 : 0)
                          : (((int)blockIdx.x < p.n_tiles) ? (p.n_tiles - 1 - (int)blockIdx.x) / p.splits + 1 : 0);
    auto tile_of = [&](int k) { return walk ? 0 : (int)blockIdx.x + k * p.splits; };
    auto head_of = [&](int k) { return walk ? (int)blockIdx.x + k * p.walk_ctas : (int)blockIdx.y; };
    auto issue_weights = [&](uint32_t ld, int h) {   // barrier n completes when weight block n has landed
#pragma unroll 1
        for (int n = 0; n < 4; ++n) {
            mbar_arrive_expect_tx_if(ld, &w_full[n], W_BYTES / 4);
            tma_load_3d_if(ld, sW + n * 32768, &tm_w, &w_full[n], 0, n * 128, h);
            tma_load_3d_if(ld, sW + n * 32768 + 16384, &tm_w, &w_full[n], 64, n * 128, h);
        }
    };

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < 6; ++i) mbar_init(&w_full[i], 1);
            mbar_init(acc_empty, 128);
            *abort_flag = 0;
            fence_mbar_init();
        }
        __syncwarp();
        if (n_my > 0) {
            const uint32_t ld = elect_one() ? 1u : 0u;
            // the first query tile and the weights, all at once
            mbar_arrive_expect_tx_if(ld, q_full, A_BYTES);
            tma_load_3d_if(ld, sA, &tm_q, q_full, 0, head_of(0), tile_of(0) * 128);
            tma_load_3d_if(ld, sA + 16384, &tm_q, q_full, 64, head_of(0), tile_of(0) * 128);
            issue_weights(ld, head_of(0));
        }
    }
    if (warp == 1) tmem_alloc(tmem_holder, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_holder, 0);

    int q_issued = n_my > 0 ? 1 : 0;   // producer warp: query tiles issued, for the abort path
    if (warp == 0) {
        // the remaining items: item k goes into the buffers once the products of item k - 1 have read them (walk mode:
        // the next head's weights as well)
        const uint32_t ld = elect_one() ? 1u : 0u;
        for (int k = 1; k < n_my; ++k) {
            if (!mbar_wait_warp(acc_full, (k - 1) & 1, abort_flag)) break;
            mbar_arrive_expect_tx_if(ld, q_full, A_BYTES);
            tma_load_3d_if(ld, sA, &tm_q, q_full, 0, head_of(k), tile_of(k) * 128);
            tma_load_3d_if(ld, sA + 16384, &tm_q, q_full, 64, head_of(k), tile_of(k) * 128);
            if (walk) issue_weights(ld, head_of(k));
            q_issued = k + 1;
        }
    } else if (warp == 1) {
        const uint32_t ld = elect_one() ? 1u : 0u;
        constexpr uint32_t idesc = idesc_bf16(128, 128, false, false);
        bool ok = true;
        for (int k = 0; k < n_my && ok; ++k) {
            ok = mbar_wait_warp(q_full, k & 1, abort_flag);
            if (ok && k > 0) ok = mbar_wait_warp(acc_empty, (k - 1) & 1, abort_flag);   // accumulators drained
            if (!ok) break;
            tc_fence_after();
            for (int n = 0; n < 4 && ok; ++n) {
                if (k == 0 || walk) {
                    ok = mbar_wait_warp(&w_full[n], walk ? (k & 1) : 0, abort_flag);
                    if (!ok) break;
                }
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
                    const uint64_t da = smem_desc_k_sw128(smem_u32(sA + ks * 16384));
                    const uint64_t db = smem_desc_k_sw128(smem_u32(sW + n * 32768 + ks * 16384));
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) umma_ss_if(ld, tmem_base + n * 128, da + 2 * kk, db + 2 * kk, idesc, (ks | kk) != 0);
                }
            }
            if (ok) umma_commit_if(ld, acc_full);
        }
    } else {
        // ---------------- epilogue: thread = one request row of the tile (tensor-memory lane)
        const int lg = (warp & 3) * 32;
        const int row = lg + lane;
        const bool leader = threadIdx.x == 64;    // first epilogue thread: issues the bulk stores
        bool ok = true;
        int blk = 0;                              // result blocks staged so far (selects the staging buffer)
        for (int k = 0; k < n_my && ok; ++k) {
            ok = __all_sync(0xffffffffu, mbar_wait(acc_full, k & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const int b0 = tile_of(k) * 128;
            const int h = head_of(k);
            if (p.B <= 32) {
                // A handful of requests (one warp's rows at most): the staged store's two block-wide barriers per
                // result block cost more than they save; every thread writes its own row.
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.q_abs) + ((int64_t)(b0 + row) * p.H + h) * 512;
#pragma unroll 1
                for (int c = 0; c < 16; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)lg << 16) + c * 32, r);
                    tmem_ld_wait();
                    if (b0 + row < p.B) {
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
                tc_fence_before();
                mbar_arrive(acc_empty);
                continue;
            }
#pragma unroll 1
            for (int n = 0; n < 4; ++n, ++blk) {
                uint8_t* stage = sOut + (blk & 1) * STAGE_BYTES;
                // the store that read this staging buffer two blocks ago must have finished reading it
                if (leader) bulk_wait_read_n<1>();
                asm volatile("bar.sync 1, 128;\n" ::: "memory");
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)lg << 16) + n * 128 + c * 32, r);
                    tmem_ld_wait();
                    // 32 columns = 64 bytes of this row in slab c / 2: 16-byte chunks (c & 1) * 4 + j, swizzled by row
                    uint8_t* srow = stage + (c >> 1) * 16384 + row * 128;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(r[j * 8 + 0]), __uint_as_float(r[j * 8 + 1]));
                        v.y = pack_bf16(__uint_as_float(r[j * 8 + 2]), __uint_as_float(r[j * 8 + 3]));
                        v.z = pack_bf16(__uint_as_float(r[j * 8 + 4]), __uint_as_float(r[j * 8 + 5]));
                        v.w = pack_bf16(__uint_as_float(r[j * 8 + 6]), __uint_as_float(r[j * 8 + 7]));
                        const int ch = ((c & 1) * 4 + j) ^ (row & 7);
                        *reinterpret_cast<uint4*>(srow + ch * 16) = v;
                    }
                }
                if (n == 3) {   // all four blocks of this tile have left tensor memory
                    tc_fence_before();
                    mbar_arrive(acc_empty);
                }
                fence_proxy_async();
                asm volatile("bar.sync 1, 128;\n" ::: "memory");
                if (leader) {
                    tma_store_3d(&tm_out, stage, n * 128, h, b0);
                    tma_store_3d(&tm_out, stage + 16384, n * 128 + 64, h, b0);
                    bulk_commit();
                }
            }
        }
        if (leader) bulk_wait_read_n<0>();   // the staging buffers must outlive the stores; the kernel end publishes the writes
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // A wait gave up: the copies that can still be in flight are the weight blocks and the query tile issued last;
        // wait for them (with a limit) before the shared memory is released, then report.
        if (warp == 0 && n_my > 0) {
            for (int n = 0; n < 4; ++n) mbar_drain(&w_full[n], walk ? (q_issued - 1) & 1 : 0);
            mbar_drain(q_full, (q_issued - 1) & 1);
        }
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

cudaError_t launch_q_absorb_sm100(const void* q_nope, const CUtensorMap* tm_w, void* q_abs, int B, int H, int n_sm, int walk_ctas, int* status,
                                  const int32_t* seq_lens, int32_t* order, const int32_t* block_table, int max_pages,
                                  int page_size, int32_t* desc, cudaStream_t s) {
    if (B <= 0) return cudaSuccess;
    CUtensorMap tm_q, tm_out;
    {
        uint64_t dims[3] = {128, (uint64_t)H, (uint64_t)B};
        uint64_t str[2] = {128 * 2, (uint64_t)H * 128 * 2};
        uint32_t box[3] = {64, 1, 128};
        cudaError_t e = make_tmap_bf16(&tm_q, q_nope, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        uint64_t dims[3] = {512, (uint64_t)H, (uint64_t)B};
        uint64_t str[2] = {512 * 2, (uint64_t)H * 512 * 2};
        uint32_t box[3] = {64, 1, 128};
        cudaError_t e = make_tmap_bf16(&tm_out, q_abs, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    const bool with_order = seq_lens != nullptr && order != nullptr && B <= 4096;
    const int n_tiles = (B + 127) / 128;
    // one CTA per head keeps the head's weights resident over all of its request tiles; with more SMs than heads
    // the tiles of a head are dealt to several CTAs
    const int splits = std::max(1, std::min(n_tiles, std::max(n_sm, 1) / H));
    // walk mode only with one request tile per head and fewer working CTAs than heads
    const int walk = (n_tiles == 1 && walk_ctas > 0 && walk_ctas < H) ? walk_ctas : 0;
    QAbsorbParams p{q_abs, B, H, n_tiles, splits, walk, status, seq_lens, order, block_table, max_pages, page_size,
                    (with_order && block_table != nullptr) ? reinterpret_cast<int4*>(desc) : nullptr};
    const dim3 grid = walk ? dim3(walk + (with_order ? 1 : 0), 1, 1) : dim3(splits, H + (with_order ? 1 : 0), 1);
    return launch_pdl(q_absorb_sm100_kernel, grid, dim3(192), SMEM_BYTES, s, tm_q, *tm_w, tm_out, p);
}

}  // namespace tmla
