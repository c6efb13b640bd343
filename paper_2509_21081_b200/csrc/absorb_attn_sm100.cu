// Absorb attention over latent tokens (Algorithm 1 line 6) on tcgen05 / TMEM / TMA.
//
// Work item (CTA) = (64 query rows, KV chunk).  Over a request's own suffix the rows are 64 heads of that
// request.  Over the shared prefix (absorb-only steps) every request attends to the same tokens, so the rows are
// 64 consecutive rows of the stacked [B * H] query matrix: with fewer than 64 heads per request (a head-sharded
// model) several requests fill one tile instead of each padding its own.  The problem is run
// transposed so that the 64 x 512 latent accumulator fits tensor memory:
//     S^T [64 tokens, 64 heads] = KV_tile [64, 576] * Q_g^T [576, 64]
//     O^T [512 latent, 64 heads] += C_tile^T [512, 64 tokens] * P^T [64 tokens, 64 heads]
// with KV_tile = [latent 512 | rope 64] of one 64-token tile of the (paged) cache and
// Q_g = [Q_A | q_pe] of the head group.  The latent part of the tile is used twice
// from shared memory: K-major as the A operand of S^T, MN-major (transposed view)
// as the A operand of O^T.  P^T (bf16) is written by the softmax threads into the
// tile's rope slab, which is dead once S^T has been computed.
//
// Softmax runs over tokens, i.e. across TMEM lanes.  To avoid a cross-lane
// reduction per tile, every head column keeps a reference exponent m_ref that is
// only raised when some logit exceeds it by more than 2^8 (a rare, collective
// "rescale" event that also rescales O^T); row sums are accumulated per thread
// and reduced across lanes once, at the end of the chunk.
//
// Warp roles (384 threads): warp 0 = TMA producer (Q once, KV ring), warp 1 =
// S^T issuer and TMEM owner, warp 3 = O^T issuer, warps 4-7 / 8-11 = softmax
// warpgroup for head columns 0-31 / 32-63.  S^T uses M = 64: token row r lives in
// TMEM lane 32 (r / 16) + r % 16, i.e. in the first 16 lanes of a warp's lane
// group.  The softmax warps read it with the 16-lane fragment shape, so that all 32
// threads hold logits: two token rows and eight columns each.
//
// Tensor memory (512 columns allocated): S^T[buf] at 64 buf (2 buffers), O^T block
// m (128 latent rows x 64 heads) at 128 + 64 m.
#include <algorithm>
#include <cstddef>

#include "kernels.h"
#include "sm100.cuh"



namespace tmla {
namespace {

using namespace sm100;

constexpr int TOK = 64;
constexpr int SLAB_BYTES = 64 * 64 * 2;          // [64 rows][64 bf16], 128-byte swizzled rows
constexpr int TILE_BYTES = 9 * SLAB_BYTES;       // 8 latent slabs + 1 rope slab = 72 KB
constexpr int STAGES = 2;
constexpr float kRescaleThreshold = 8.f;         // log2 units


struct AbsorbSm100Params {
    int B, H;
    int chunk, n_shared_chunks, n_suffix_chunks;
    int shared_groups;     // row groups per shared-prefix chunk
    int stacked;           // shared-prefix row groups cut from the stacked [B * H] query matrix (else per request)
    int Ls_absorb;
    int page_size, max_pages;
    int num_pages;         // physical pages of the paged cache: ids outside [0, num_pages) are not dereferenced
    const int32_t* block_table;
    const int32_t* seq_lens;
    const int32_t* order;
    const int4* desc;      // optional, per launch position: {request, clamped suffix length, page 0, page 1}
    float scale_log2;
    float* o_part;     // [n_chunks][B][H][512]
    float* lse_part;   // [n_chunks][B][H]
    // single-chunk launches write the merged result directly and skip the merge step
    __nv_bfloat16* o_lat_direct;   // bf16 [B][H][512] or null
    float* lse_direct;             // [B][H]
    int* status;
};

struct Shared {
    uint64_t q_full;
    // A KV tile is loaded, consumed and released in four slab groups: group g = latent slabs 2g and
    // 2g+1 (the latent rows of accumulator block g), group 3 also holds the rope slab (which becomes
    // P^T).  The logits product starts on the first group while the others are still in flight, and a
    // group is refilled as soon as its accumulator block has read it.
    uint64_t kv_full[STAGES][4], kv_empty[STAGES][4];
    uint64_t s_ready[2], p_ready[2];
    // completion of the accumulation of tile j goes to o_done[j & 1]: a waiter that knows tile j-2 has
    // landed (every wait below does) then sees a barrier at most one completion from the awaited one,
    // which is what a parity wait can tell apart
    uint64_t o_done[2];
    uint32_t tmem_base;
    int abort_flag;
    float red[2][4][32];   // [warpgroup][warp][column]: cross-warp reductions
    float mref[2][32];     // [warpgroup][column]: reference exponent (log2 units) of each head column
    alignas(16) float inv[2][32];   // [warpgroup][column]: inverse row sums for the epilogue
};

constexpr int kAbsorbSmem = (STAGES + 1) * TILE_BYTES + 1024 + (int)sizeof(Shared) + 64;

__device__ __forceinline__ bool wg_vote_or(int bar_id, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n.reg .pred p, q;\nsetp.ne.b32 q, %2, 0;\n"
        "bar.red.or.pred p, %1, 128, q;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(r) : "r"(bar_id), "r"(pred ? 1u : 0u) : "memory");
    return r != 0;
}
__device__ __forceinline__ void wg_sync(int bar_id) { asm volatile("bar.sync %0, 128;\n" ::"r"(bar_id) : "memory"); }

__global__ void __launch_bounds__(384, 1)
absorb_attn_sm100_kernel(const __grid_constant__ CUtensorMap tm_qa, const __grid_constant__ CUtensorMap tm_qp,
                         const __grid_constant__ CUtensorMap tm_ckv_sh, const __grid_constant__ CUtensorMap tm_kpe_sh,
                         const __grid_constant__ CUtensorMap tm_ckv_pg, const __grid_constant__ CUtensorMap tm_kpe_pg,
                         AbsorbSm100Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sKV = smem;                                  // STAGES tiles
    uint8_t* sQ = smem + STAGES * TILE_BYTES;             // 9 slabs [64 heads][64]
    Shared* sh = reinterpret_cast<Shared*>(sQ + TILE_BYTES);
    volatile int* abort_flag = &sh->abort_flag;

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    pdl_trigger();
    pdl_wait();   // the descriptors and Q_A read below are written by the preceding kernel
    // Work items in launch order: the shared-prefix items (chunk fastest, then row group), then the suffix items
    // (chunk fastest, then head group, then request position in longest-first order).
    const int n_shared_items = p.n_shared_chunks * p.shared_groups;
    const bool shared_seg = (int)blockIdx.x < n_shared_items;
    int chunk, row0, n_rows, b = 0, len_b = -1, pg0 = -1, pg1 = -1;
    if (shared_seg) {
        chunk = blockIdx.x % p.n_shared_chunks;
        const int g = blockIdx.x / p.n_shared_chunks;
        if (p.stacked) {                       // 64 consecutive rows of the stacked query matrix
            row0 = g * 64;
            n_rows = min(64, p.B * p.H - row0);
        } else {                               // 64 heads of one request
            const int hg = (p.H + 63) / 64;
            b = g / hg;
            row0 = b * p.H + (g % hg) * 64;
            n_rows = min(64, p.H - (g % hg) * 64);
        }
    } else {
        const int i = blockIdx.x - n_shared_items, hg = (p.H + 63) / 64;
        chunk = p.n_shared_chunks + i % p.n_suffix_chunks;
        const int y = (i / p.n_suffix_chunks) % hg, z = i / (p.n_suffix_chunks * hg);
        // one 16-byte load gives the request, its suffix length and its first two pages (else three
        // dependent loads stand between the kernel's start and its first copy)
        if (p.desc != nullptr) {
            const int4 d = p.desc[z];
            b = d.x; len_b = d.y; pg0 = d.z; pg1 = d.w;
        } else {
            b = p.order ? p.order[z] : z;
        }
        row0 = b * p.H + y * 64;
        n_rows = min(64, p.H - y * 64);
    }

    // token range of this chunk
    int seg_len, tok_begin;
    if (shared_seg) {
        seg_len = p.Ls_absorb;
        tok_begin = chunk * p.chunk;
    } else {
        seg_len = len_b >= 0 ? len_b : min(max(p.seq_lens[b], 0), p.max_pages * p.page_size);
        tok_begin = (chunk - p.n_shared_chunks) * p.chunk;
    }
    const int tok_end = min(seg_len, tok_begin + p.chunk);
    const int n_tiles = tok_end > tok_begin ? (tok_end - tok_begin + TOK - 1) / TOK : 0;

    // Warp 0 initialises the barriers and at once issues the Q load and the first tiles, so that the
    // first copies are in flight while the rest of the CTA sets up (tensor-memory allocation, barrier).
    const CUtensorMap* tc = shared_seg ? &tm_ckv_sh : &tm_ckv_pg;
    const CUtensorMap* tk = shared_seg ? &tm_kpe_sh : &tm_kpe_pg;
    const int32_t* bt = p.block_table + (int64_t)b * p.max_pages;
    const uint32_t ld0 = (warp == 0 && elect_one()) ? 1u : 0u;
    // physical page and slot of tile j (the block-table read is issued ahead of the wait for a free
    // ring slot so that its latency is off the critical path)
    bool bad_page = false;   // producer warp only: a page id of the caller's table was out of range
    auto page_of = [&](int j, int& page, int& slot) {
        const int t0 = tok_begin + j * TOK;
        if (shared_seg) {
            page = t0 / TOK;
            slot = 0;
        } else {
            const int idx = t0 / p.page_size;
            page = (p.desc != nullptr && idx < 2) ? (idx == 0 ? pg0 : pg1) : __shfl_sync(0xffffffffu, bt[idx], 0);
            slot = t0 % p.page_size;
            // The tensor map ends at num_pages: a coordinate at or past it reads as zeros instead of touching
            // memory the caller does not own.  The violation is reported through the status word.
            if ((unsigned)page >= (unsigned)p.num_pages) {
                bad_page = true;
                page = p.num_pages;
            }
        }
    };
    auto issue_group = [&](int j, int g, int page, int slot) {
        const int s = j & 1;
        uint8_t* dst = sKV + s * TILE_BYTES;
        mbar_arrive_expect_tx_if(ld0, &sh->kv_full[s][g], (g == 3 ? 3 : 2) * SLAB_BYTES);
        tma_load_3d_if(ld0, dst + (2 * g) * SLAB_BYTES, tc, &sh->kv_full[s][g], (2 * g) * 64, slot, page);
        tma_load_3d_if(ld0, dst + (2 * g + 1) * SLAB_BYTES, tc, &sh->kv_full[s][g], (2 * g + 1) * 64, slot, page);
        if (g == 3) tma_load_3d_if(ld0, dst + 8 * SLAB_BYTES, tk, &sh->kv_full[s][g], 0, slot, page);
    };
    // The ring holds two tiles, so the load of tile j + 2 can only start when tile j has been consumed and its
    // latency (1.5-2 us from DRAM) is exposed once per pair of tiles.  Tile j + 2 is therefore requested into L2
    // when tile j's loads go out; the load into the freed slot then completes in an L2 round trip.
    // (Measured: 2-3 % on long ragged suffixes that keep HBM saturated; nothing or slightly negative for chunks of
    // a few tiles and for the shared prefix in absorb-only mode, whose tiles every request re-reads from L2 anyway;
    // those skip it.)
    const bool use_prefetch = n_tiles > 8 && !shared_seg;
    auto prefetch_tile = [&](int j) {
        if (!use_prefetch || j >= n_tiles) return;
        int page, slot;
        page_of(j, page, slot);
#pragma unroll 1
        for (int sl = 0; sl < 8; ++sl) tma_prefetch_3d_if(ld0, tc, sl * 64, slot, page);
        tma_prefetch_3d_if(ld0, tk, 0, slot, page);
    };
    if (warp == 2) {   // otherwise idle: fetch the tensor maps while warp 0 sets up the barriers
        if (lane == 0) prefetch_tmap(&tm_qa);
        if (lane == 1) prefetch_tmap(&tm_qp);
        if (lane == 2) prefetch_tmap(tc);
        if (lane == 3) prefetch_tmap(tk);
    }
    if (warp == 0) {
        // the mbarriers are the leading uint64_t members of the struct, one lane each; p_ready counts the
        // 256 softmax threads, all others one arrival
        uint64_t* all = &sh->q_full;
        constexpr int n_bars = (int)(offsetof(Shared, tmem_base) / sizeof(uint64_t));
        for (int i = lane; i < n_bars; i += 32) {
            uint64_t* m = all + i;
            mbar_init(m, (m >= &sh->p_ready[0] && m < &sh->o_done[0]) ? 256 : 1);
        }
        if (lane == 0) sh->abort_flag = 0;
        fence_mbar_init();
        __syncwarp();
        if (n_tiles > 0) {
            mbar_arrive_expect_tx_if(ld0, &sh->q_full, TILE_BYTES);
#pragma unroll 1
            for (int s = 0; s < 8; ++s) tma_load_2d_if(ld0, sQ + s * SLAB_BYTES, &tm_qa, &sh->q_full, s * 64, row0);
            tma_load_2d_if(ld0, sQ + 8 * SLAB_BYTES, &tm_qp, &sh->q_full, 0, row0);
            for (int j = 0; j < min(n_tiles, STAGES); ++j) {
                int page, slot;
                page_of(j, page, slot);
#pragma unroll 1
                for (int g = 0; g < 4; ++g) issue_group(j, g, page, slot);
            }
            for (int j = STAGES; j < 2 * STAGES; ++j) prefetch_tile(j);
        }
    }
    if (warp == 1) tmem_alloc(&sh->tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, sh->tmem_base, 0);

    int tiles_issued = min(n_tiles, STAGES);   // producer warp: tiles whose copies were issued (upper bound), for the abort path
    if (n_tiles > 0) {
        if (warp == 0) {
            // ---------------- producer: the rest of the KV ring (Q and the first tiles are already in flight)
            for (int j = STAGES; j < n_tiles; ++j) {
                tiles_issued = j + 1;
                int page, slot;
                page_of(j, page, slot);
                bool ok = true;
#pragma unroll 1
                for (int g = 0; g < 4 && ok; ++g) {
                    ok = mbar_wait_warp(&sh->kv_empty[j & 1][g], ((j >> 1) & 1) ^ 1, abort_flag);
                    if (ok) issue_group(j, g, page, slot);
                }
                if (!ok) break;
                prefetch_tile(j + STAGES);
            }
        } else if (warp == 1) {
            // ---------------- S^T = KV_tile * Q^T issuer (M = 64 tokens, N = 64 heads, K = 576)
            const uint32_t ld = elect_one() ? 1u : 0u;
            constexpr uint32_t idesc_s = idesc_bf16(64, 64, false, false);
            bool ok = mbar_wait_warp(&sh->q_full, 0, abort_flag);
            const uint32_t qa = smem_u32(sQ);
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int s = j & 1;
                if (j >= 2) {   // the softmax of tile j-2 has finished reading this S^T buffer
                    ok = mbar_wait_warp(&sh->p_ready[s], ((j >> 1) - 1) & 1, abort_flag);
                    if (!ok) break;
                }
                const uint32_t ka = smem_u32(sKV + s * TILE_BYTES);
                const uint32_t d = tmem_base + (uint32_t)(s * 64);
                // the contraction over the 576 dims runs group by group as the slabs land
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    ok = mbar_wait_warp(&sh->kv_full[s][g], (j >> 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int i = 0; i < 3; ++i) {
                        if (i == 2 && g != 3) continue;
                        const int sl = (i == 2) ? 8 : 2 * g + i;
                        const uint64_t da = smem_desc_k_sw128(ka + sl * SLAB_BYTES);
                        const uint64_t db = smem_desc_k_sw128(qa + sl * SLAB_BYTES);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_ss_if(ld, d, da + 2 * k, db + 2 * k, idesc_s, (g | i | k) != 0);
                    }
                }
                if (!ok) break;
                umma_commit_if(ld, &sh->s_ready[s]);
            }
        } else if (warp == 3) {
            // ---------------- O^T += C^T * P^T issuer (4 blocks of M = 128 latent rows, N = 64 heads, K = 64 tokens)
            const uint32_t ld = elect_one() ? 1u : 0u;
            constexpr uint32_t idesc_o = idesc_bf16(128, 64, true, true);
            bool ok = true;
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int s = j & 1;
                ok = mbar_wait_warp(&sh->p_ready[s], (j >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t ca = smem_u32(sKV + s * TILE_BYTES);
                const uint32_t pa = ca + 8 * SLAB_BYTES;     // P^T lives in the rope slab
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const uint32_t d = tmem_base + 128u + (uint32_t)m * 64u;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t da = smem_desc_mn_sw128(ca + (2 * m) * SLAB_BYTES + k * 2048, SLAB_BYTES, 1024);
                        const uint64_t db = smem_desc_mn_sw128(pa + k * 2048, SLAB_BYTES, 1024);
                        umma_ss_if(ld, d, da, db, idesc_o, (j | k) != 0);
                    }
                    // accumulator block m was the last reader of latent slabs 2m, 2m+1 (and, for m = 3, of P^T)
                    umma_commit_if(ld, &sh->kv_empty[s][m]);
                }
                umma_commit_if(ld, &sh->o_done[s]);
            }
        } else if (warp >= 4) {
            // ---------------- softmax warpgroups
            const int cg = (warp - 4) >> 2;                 // column group: query rows row0 + 32 cg .. + 31
            const int q = warp & 3;                         // TMEM lane quadrant of this warp
            const int bar_id = 1 + cg;
            // S^T has M = 64: the 16 token rows of this warp's quadrant sit in its first 16 tensor-memory lanes.  They
            // are read as fragments so that all 32 threads work: thread t holds, for the tokens ra = 16 q + t/4 and
            // rb = ra + 8, the logits of the columns 8g + 2(t%4) + {0, 1} (g = 0..3) of this warpgroup's 32 columns.
            const int qq = lane & 3;
            const int ra = 16 * q + (lane >> 2), rb = ra + 8;
            const uint32_t lane_base = (uint32_t)(32 * q) << 16;
            // Per-thread state: partial sums of this thread's eight columns over its two token rows.  The reference
            // exponents are the same for every thread of the warpgroup and live in shared memory.
            float l_part[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) l_part[c] = 0.f;
            volatile float* mref = sh->mref[cg];
            if (q == 0) mref[lane] = -INFINITY;
            wg_sync(bar_id);
            float neg_mr[8];       // register copy of -m_ref of this thread's columns, refreshed after every rescale event
#pragma unroll
            for (int c = 0; c < 8; ++c) neg_mr[c] = INFINITY;

            for (int j = 0; j < n_tiles; ++j) {
                const int s = j & 1;
                bool ok = __all_sync(0xffffffffu, mbar_wait(&sh->s_ready[s], (j >> 1) & 1, abort_flag));
                const int t0 = tok_begin + j * TOK;
                const int n_valid = min(TOK, tok_end - t0);
                uint32_t sr[16], pka[4], pkb[4];   // logits; packed probabilities of row a / row b (columns 8g+2qq, +1)
                bool exceed = false;
                if (ok) {
                    tc_fence_after();
                    tmem_ld_16x256b_x4(tmem_base + lane_base + (uint32_t)(s * 64 + cg * 32), sr);
                    tmem_ld_wait();
                    // one pass: distance of the scaled logit to the reference (one FMA), probability
                    // (speculative: final unless the warpgroup votes for a rescale).  Token rows past the end
                    // carry -inf.
                    if (ra >= n_valid) {
#pragma unroll
                        for (int g = 0; g < 4; ++g) sr[4 * g] = sr[4 * g + 1] = 0xff800000u;
                    }
                    if (rb >= n_valid) {
#pragma unroll
                        for (int g = 0; g < 4; ++g) sr[4 * g + 2] = sr[4 * g + 3] = 0xff800000u;
                    }
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const float a0 = fmaf(__uint_as_float(sr[4 * g]), p.scale_log2, neg_mr[2 * g]);
                        const float a1 = fmaf(__uint_as_float(sr[4 * g + 1]), p.scale_log2, neg_mr[2 * g + 1]);
                        const float b0 = fmaf(__uint_as_float(sr[4 * g + 2]), p.scale_log2, neg_mr[2 * g]);
                        const float b1 = fmaf(__uint_as_float(sr[4 * g + 3]), p.scale_log2, neg_mr[2 * g + 1]);
                        exceed |= (a0 > kRescaleThreshold) | (a1 > kRescaleThreshold) | (b0 > kRescaleThreshold) | (b1 > kRescaleThreshold);
                        pka[g] = pack_bf16(fast_exp2(a0), fast_exp2(a1));
                        pkb[g] = pack_bf16(fast_exp2(b0), fast_exp2(b1));
                    }
                }
                const bool rescale = wg_vote_or(bar_id, exceed);
                if (*abort_flag) break;                      // uniform across the warpgroup after the barrier
                if (rescale) {
                    // exact column maxima of this tile across the 64 token rows: over this thread's two rows, then
                    // over the eight threads of the warp that hold the same columns (lanes t%4 equal), then across the
                    // four warps through shared memory
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int g = c >> 1, e = c & 1;
                        float v = fmaxf(__uint_as_float(sr[4 * g + e]), __uint_as_float(sr[4 * g + 2 + e])) * p.scale_log2;
                        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
                        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
                        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 16));
                        if (lane < 4) sh->red[cg][q][8 * g + 2 * qq + e] = v;
                    }
                    wg_sync(bar_id);
                    const float cm = fmaxf(fmaxf(sh->red[cg][0][lane], sh->red[cg][1][lane]), fmaxf(sh->red[cg][2][lane], sh->red[cg][3][lane]));
                    const float m_old = mref[lane];
                    const float m_new = fmaxf(m_old, cm);
                    const float f_lane = (m_new == -INFINITY) ? 1.f : fast_exp2(m_old - m_new);   // factor of column `lane`
                    wg_sync(bar_id);                         // everyone has read the old references
                    if (q == 0) mref[lane] = m_new;
                    wg_sync(bar_id);
#pragma unroll
                    for (int c = 0; c < 8; ++c) l_part[c] *= __shfl_sync(0xffffffffu, f_lane, 8 * (c >> 1) + 2 * qq + (c & 1));
                    if (j > 0) {
                        // rescale this column group's 32 columns of all four O^T blocks (all 128 lanes), once
                        // the previous tile's accumulation has landed
                        mbar_wait(&sh->o_done[(j - 1) & 1], ((j - 1) >> 1) & 1, abort_flag);
                        __syncwarp();
                        tc_fence_after();
#pragma unroll 1
                        for (int m = 0; m < 4; ++m) {
                            uint32_t orr[32];
                            const uint32_t o_addr = tmem_base + lane_base + 128u + (uint32_t)(m * 64 + cg * 32);
                            tmem_ld32(o_addr, orr);
                            tmem_ld_wait();
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                orr[c] = __float_as_uint(__uint_as_float(orr[c]) * __shfl_sync(0xffffffffu, f_lane, c));
                            tmem_st32(o_addr, orr);
                        }
                        tmem_st_wait();
                    }
                    // probabilities again, against the new references
#pragma unroll
                    for (int c = 0; c < 8; ++c) neg_mr[c] = -mref[8 * (c >> 1) + 2 * qq + (c & 1)];
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        pka[g] = pack_bf16(fast_exp2(fmaf(__uint_as_float(sr[4 * g]), p.scale_log2, neg_mr[2 * g])),
                                           fast_exp2(fmaf(__uint_as_float(sr[4 * g + 1]), p.scale_log2, neg_mr[2 * g + 1])));
                        pkb[g] = pack_bf16(fast_exp2(fmaf(__uint_as_float(sr[4 * g + 2]), p.scale_log2, neg_mr[2 * g])),
                                           fast_exp2(fmaf(__uint_as_float(sr[4 * g + 3]), p.scale_log2, neg_mr[2 * g + 1])));
                    }
                }
                // per-thread partial column sums (of the bf16-rounded values), P^T into the rope slab
                uint8_t* tile = sKV + s * TILE_BYTES;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    l_part[2 * g] += __uint_as_float(pka[g] << 16) + __uint_as_float(pkb[g] << 16);
                    l_part[2 * g + 1] += __uint_as_float(pka[g] & 0xffff0000u) + __uint_as_float(pkb[g] & 0xffff0000u);
                    // MN-major P^T: row (token) = 64 heads = 128 bytes, 16-byte chunks swizzled by row & 7; this
                    // thread's column pair is word qq of chunk cg * 4 + g (the four threads of a row fill the chunk)
                    const int ch = cg * 4 + g;
                    *reinterpret_cast<uint32_t*>(tile + 8 * SLAB_BYTES + ra * 128 + ((ch ^ (ra & 7)) * 16) + qq * 4) = pka[g];
                    *reinterpret_cast<uint32_t*>(tile + 8 * SLAB_BYTES + rb * 128 + ((ch ^ (rb & 7)) * 16) + qq * 4) = pkb[g];
                }
                if (n_valid < TOK) {
                    // ragged tail: latent rows of tokens past the end may hold anything (even NaN);
                    // zero them so that 0 * garbage cannot reach the accumulator
                    const int tid_sm = threadIdx.x - 128;
                    const int n_chunks16 = (TOK - n_valid) * 64;             // 8 slabs x 8 chunks per row
                    for (int idx = tid_sm; idx < n_chunks16; idx += 256) {
                        const int row = n_valid + idx / 64, rem = idx % 64;
                        *reinterpret_cast<uint4*>(tile + (rem >> 3) * SLAB_BYTES + row * 128 + (rem & 7) * 16) = make_uint4(0, 0, 0, 0);
                    }
                }
                fence_proxy_async();
                tc_fence_before();
                mbar_arrive(&sh->p_ready[s]);
            }

            // ---------------- epilogue: row sums across lanes, normalised partial, LSE
            // (the decision to run it is taken by a warpgroup vote so that every thread of the
            // warpgroup reaches the same named barriers)
            bool staged = false;
            if (!wg_vote_or(bar_id, *abort_flag != 0)) {
                // Column sums first (they do not depend on the accumulator, whose last product is still running):
                // over the eight threads of the warp that hold the same columns, then the four warps add up through
                // shared memory.
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    float v = l_part[c];
                    v += __shfl_xor_sync(0xffffffffu, v, 4);
                    v += __shfl_xor_sync(0xffffffffu, v, 8);
                    v += __shfl_xor_sync(0xffffffffu, v, 16);
                    if (lane < 4) sh->red[cg][q][8 * (c >> 1) + 2 * qq + (c & 1)] = v;
                }
                wg_sync(bar_id);
                if (q == 0) {   // lane = head column: its inverse row sum and LSE
                    const float l = sh->red[cg][0][lane] + sh->red[cg][1][lane] + sh->red[cg][2][lane] + sh->red[cg][3][lane];
                    sh->inv[cg][lane] = 1.f / l;
                    const int r = cg * 32 + lane;
                    if (r < n_rows) {
                        const float lse = (mref[lane] + log2f(l)) * kLn2;
                        if (p.o_lat_direct) p.lse_direct[row0 + r] = lse;
                        else p.lse_part[(int64_t)chunk * p.B * p.H + row0 + r] = lse;
                    }
                }
                wg_sync(bar_id);
                float inv[32];
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    const float4 v = *reinterpret_cast<const float4*>(&sh->inv[cg][c]);
                    inv[c] = v.x; inv[c + 1] = v.y; inv[c + 2] = v.z; inv[c + 3] = v.w;
                }
                const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh->o_done[(n_tiles - 1) & 1], ((n_tiles - 1) >> 1) & 1, abort_flag));
                tc_fence_after();
                if (ok && !*abort_flag) {
                    // The normalised O (head-major rows of 512 latent values) is staged in the KV ring, which
                    // no product reads any more, as the contiguous block of up to 64 head rows it forms in
                    // global memory, and leaves with one bulk copy.
                    const bool direct = p.o_lat_direct != nullptr;
#pragma unroll 1
                    for (int m = 0; m < 4; ++m) {
                        uint32_t orr[32];
                        tmem_ld32(tmem_base + lane_base + 128u + (uint32_t)(m * 64 + cg * 32), orr);
                        tmem_ld_wait();
                        const int lat = m * 128 + 32 * q + lane;
                        if (direct) {
                            __nv_bfloat16* st = reinterpret_cast<__nv_bfloat16*>(sKV) + (cg * 32) * 512 + lat;
#pragma unroll
                            for (int c = 0; c < 32; ++c) st[c * 512] = __float2bfloat16_rn(__uint_as_float(orr[c]) * inv[c]);
                        } else {
                            float* st = reinterpret_cast<float*>(sKV) + (cg * 32) * 512 + lat;
#pragma unroll
                            for (int c = 0; c < 32; ++c) st[c * 512] = __uint_as_float(orr[c]) * inv[c];
                        }
                    }
                    fence_proxy_async();
                    staged = true;
                }
            }
            // Both warpgroups have staged their heads, or at least one has set the abort flag (every
            // thread of the two warpgroups gets here: named barrier 3, 256 threads).
            asm volatile("bar.sync 3, 256;\n" ::: "memory");
            if (threadIdx.x == 128 && staged && !*abort_flag) {
                if (p.o_lat_direct) {
                    bulk_store(p.o_lat_direct + (int64_t)row0 * 512, sKV, (uint32_t)n_rows * 1024u);
                } else {
                    bulk_store(p.o_part + ((int64_t)chunk * p.B * p.H + row0) * 512, sKV, (uint32_t)n_rows * 2048u);
                }
                bulk_commit();
                bulk_wait_read();   // the staging buffer must outlive the copy; the kernel end publishes the writes
            }
        }
    } else if (warp >= 4) {
        // empty chunk: weight zero in the merge
        const int i = threadIdx.x - 128;
        if (i < n_rows) {
            if (p.o_lat_direct) {
                // a request without any latent token: zero latent output, weight zero in the combine
                p.lse_direct[row0 + i] = -INFINITY;
                for (int l = 0; l < 512; l += 8)
                    *reinterpret_cast<uint4*>(p.o_lat_direct + (int64_t)(row0 + i) * 512 + l) = make_uint4(0, 0, 0, 0);
            } else {
                p.lse_part[(int64_t)chunk * p.B * p.H + row0 + i] = -INFINITY;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && bad_page && p.status) atomicOr(p.status, 0x100);
    if (*abort_flag) {
        // A wait gave up.  Before the CTA's shared memory is released the producer warp waits (with a limit) on the
        // barriers of the tiles it issued last and of the query tile: only those copies can still be in flight.
        if (warp == 0 && n_tiles > 0) {
            for (int j = max(0, tiles_issued - STAGES); j < tiles_issued; ++j)
                for (int g = 0; g < 4; ++g) mbar_drain(&sh->kv_full[j & 1][g], (j >> 1) & 1);
            mbar_drain(&sh->q_full, 0);
        }
        if (threadIdx.x == 0 && p.status) atomicOr(p.status, 3);
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

cudaError_t make_kv_tmaps(const void* ckv, const void* kpe, int64_t ckv_stride, int64_t kpe_stride, int page_size,
                          uint64_t n_pages, CUtensorMap* tm_ckv, CUtensorMap* tm_kpe) {
    {
        uint64_t dims[3] = {512, (uint64_t)page_size, n_pages};
        uint64_t str[2] = {(uint64_t)ckv_stride * 2, (uint64_t)page_size * ckv_stride * 2};
        uint32_t box[3] = {64, TOK, 1};
        cudaError_t e = make_tmap_bf16(tm_ckv, ckv, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        uint64_t dims[3] = {64, (uint64_t)page_size, n_pages};
        uint64_t str[2] = {(uint64_t)kpe_stride * 2, (uint64_t)page_size * kpe_stride * 2};
        uint32_t box[3] = {64, TOK, 1};
        cudaError_t e = make_tmap_bf16(tm_kpe, kpe, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace


cudaError_t set_attrs_absorb_sm100() {
    return cudaFuncSetAttribute(absorb_attn_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAbsorbSmem);
}

cudaError_t make_absorb_shared_tmaps(const void* ckv, const void* kpe, int64_t Ls_pad, CUtensorMap* tm_ckv,
                                     CUtensorMap* tm_kpe) {
    return make_kv_tmaps(ckv, kpe, 512, 64, TOK, (uint64_t)(Ls_pad / TOK), tm_ckv, tm_kpe);
}

cudaError_t launch_absorb_attn_sm100(const AbsorbAttn& a, const CUtensorMap* tm_ckv_sh, const CUtensorMap* tm_kpe_sh,
                                     void* o_lat_direct, float* lse_direct, int* status, cudaStream_t s) {
    const int n_chunks = a.n_shared_chunks + a.n_suffix_chunks;
    if (a.B <= 0 || n_chunks <= 0) return cudaSuccess;
    if (a.chunk % TOK != 0) return cudaErrorInvalidValue;
    CUtensorMap tm_qa, tm_qp, tm_ckv_pg, tm_kpe_pg;
    {   // the queries as one [B * H, 512] matrix: a box is 64 consecutive rows (of one request or across requests);
        // rows past the end read as zeros
        uint64_t dims[2] = {512, (uint64_t)a.H * (uint64_t)a.B};
        uint64_t str[1] = {512 * 2};
        uint32_t box[2] = {64, 64};
        cudaError_t e = make_tmap_bf16(&tm_qa, a.q_abs, 2, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        uint64_t dims[2] = {64, (uint64_t)a.H * (uint64_t)a.B};
        uint64_t str[1] = {64 * 2};
        uint32_t box[2] = {64, 64};
        cudaError_t e = make_tmap_bf16(&tm_qp, a.q_pe, 2, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    if (a.n_suffix_chunks > 0) {
        // the maps end at the caller's last physical page: anything past it reads as zeros
        cudaError_t e = make_kv_tmaps(a.ckv_pages, a.kpe_pages, a.ckv_stride, a.kpe_stride, a.page_size,
                                      (uint64_t)std::max(a.num_pages, 1), &tm_ckv_pg, &tm_kpe_pg);
        if (e != cudaSuccess) return e;
    } else {
        tm_ckv_pg = *tm_ckv_sh;
        tm_kpe_pg = *tm_kpe_sh;
    }
    AbsorbSm100Params p{};
    p.B = a.B; p.H = a.H;
    p.chunk = a.chunk; p.n_shared_chunks = a.n_shared_chunks; p.n_suffix_chunks = a.n_suffix_chunks;
    const int head_groups = (a.H + 63) / 64;
    p.stacked = a.stacked ? 1 : 0;
    p.shared_groups = a.stacked ? (int)(((int64_t)a.B * a.H + 63) / 64) : a.B * head_groups;
    p.Ls_absorb = a.Ls_absorb;
    p.page_size = a.page_size; p.max_pages = a.max_pages; p.num_pages = a.num_pages;
    p.block_table = a.block_table; p.seq_lens = a.seq_lens; p.order = a.order;
    p.desc = reinterpret_cast<const int4*>(a.desc);
    p.scale_log2 = a.scale * kLog2e;
    p.o_part = a.o_part; p.lse_part = a.lse_part; p.status = status;
    p.o_lat_direct = n_chunks == 1 ? reinterpret_cast<__nv_bfloat16*>(o_lat_direct) : nullptr;
    p.lse_direct = lse_direct;
    const int smem = kAbsorbSmem;
    dim3 grid(a.n_shared_chunks * p.shared_groups + a.n_suffix_chunks * head_groups * a.B, 1, 1);
    const CUtensorMap* sh_c = a.n_shared_chunks > 0 ? tm_ckv_sh : &tm_ckv_pg;
    const CUtensorMap* sh_k = a.n_shared_chunks > 0 ? tm_kpe_sh : &tm_kpe_pg;
    return launch_pdl(absorb_attn_sm100_kernel, grid, dim3(384), smem, s, tm_qa, tm_qp, *sh_c, *sh_k, tm_ckv_pg, tm_kpe_pg, p);
}

}  // namespace tmla
