// Naive shared-prefix attention (Algorithm 1 line 4) on tcgen05 / TMEM / TMA.
//
// Per head h the step is a dense contraction over all B query rows:
//     S = Q_h [B,192] * [K_nope_h | k_pe]^T [192, L_s],  O = softmax(S) * V_h [L_s,128].
// A CTA owns one head, one group of query rows and one KV split, and runs two
// independent attention "streams" that share the TMA/MMA machinery:
//   * B > 128  (mode X, 128-token KV tiles): stream i = query rows [256g + 128i, +128);
//     both streams consume every KV tile of the split (tiles are loaded once).  This
//     is the compute-bound regime: N = 128 per S MMA halves the re-reads of Q from
//     shared memory, the two streams ping-pong between tensor core and softmax.
//   * B <= 128 (mode Y, 64-token KV tiles): both streams use the same 128 query rows;
//     stream i takes every second KV tile (tile k -> stream k & 1) with its own softmax
//     state.  This is the HBM-bound regime: small tiles give a four-deep ring per operand.
// Each stream writes a normalised fp32 partial and its LSE; the combine step merges all
// partials of a (request, head).
//
// Warp roles (384 threads): warp 0 = TMA producer for Q and the K ring, warp 2 = TMA
// producer for the V ring, warp 1 = issuer of the S = Q K^T MMAs and TMEM owner, warp 3
// = issuer of the O += P V MMAs, warps 4-7 / 8-11 = softmax warpgroup of stream 0 / 1
// (thread = one query row).  Two issuing warps keep the K-side and V-side barrier waits
// from serialising behind each other; role warps run their loops with all lanes and
// predicate the issuing instruction on one elected lane.
//
// Tensor memory (512 columns).  64-token tiles: S[i][buf] (64 fp32 columns, double
// buffered; P in bf16 overwrites the first 32) at (2i+buf)*64, O[i] at 256 + 128 i.
// 128-token tiles: S[i] (128 columns, P overwrites the first 64) at 128 i, O[i] at
// 256 + 128 i.
//
// The expanded cache is stored in 64-token blocks: K_nope [H, L/64, 2 slabs, 64, 64],
// V^T [H, L/64, 128, 64], rope keys [L, 64]; every TMA box is a contiguous 8 or 16 KB.
//
// Every mbarrier wait has a deadline; on expiry all roles fall through to the common
// teardown and the status word is set.
#include "kernels.h"
#include "sm100.cuh"

namespace tmla {
namespace {

using namespace sm100;

constexpr int Q_TILE_BYTES = 128 * 192 * 2;   // 3 slabs [128][64] bf16
constexpr int MAX_STAGES = 4;

struct NaiveSm100Params {
    int B, H, Ls, Ls_pad;
    int n_split, m_groups;
    int k_stages, v_stages;
    float scale_log2;
    float* o_part;     // [n_slots][B][H][128]
    float* lse_part;   // [n_slots][B][H]
    int* status;
};

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[MAX_STAGES], k_empty[MAX_STAGES];
    uint64_t v_full[MAX_STAGES], v_empty[MAX_STAGES];
    uint64_t s_ready[2][2], p_ready[2][2], sbuf_free[2][2], o_done[2];
    uint32_t tmem_base;
    int abort_flag;
};

// TOK = tokens per KV tile: 64 (mode Y, B <= 128) or 128 (mode X, B > 128).
template <int TOK>
__global__ void __launch_bounds__(384, 1)
naive_attn_sm100_kernel(const __grid_constant__ CUtensorMap tm_qn, const __grid_constant__ CUtensorMap tm_qp,
                        const __grid_constant__ CUtensorMap tm_kn, const __grid_constant__ CUtensorMap tm_kp,
                        const __grid_constant__ CUtensorMap tm_vt, NaiveSm100Params p) {
    constexpr bool MODE_Y = TOK == 64;
    constexpr int NB = MODE_Y ? 2 : 1;                  // S buffers per stream
    constexpr int BLK = TOK / 64;                       // 64-token blocks per tile
    constexpr int K_SLAB = TOK * 128;                   // bytes of one [TOK][64] K slab
    constexpr int K_TILE_BYTES = 3 * K_SLAB;
    constexpr int V_TILE_BYTES = BLK * 16384;           // BLK slabs [128 dims][64 tokens]

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int n_q_tiles = MODE_Y ? 1 : 2;
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + n_q_tiles * Q_TILE_BYTES;
    uint8_t* sV = sK + p.k_stages * K_TILE_BYTES;
    Barriers* bar = reinterpret_cast<Barriers*>(sV + p.v_stages * V_TILE_BYTES);
    volatile int* abort_flag = &bar->abort_flag;

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    const int split = blockIdx.x / p.m_groups, mg = blockIdx.x % p.m_groups, h = blockIdx.y;
    const int row0 = mg * (MODE_Y ? 128 : 256);

    // KV tiles of this split
    const int n_tiles_total = (p.Ls + TOK - 1) / TOK;
    const int per = (n_tiles_total + p.n_split - 1) / p.n_split;
    const int t_begin = split * per;
    const int t_end = min(n_tiles_total, t_begin + per);
    const int n_tiles = max(t_end - t_begin, 0);
    // tiles per stream and number of steps
    int n_str[2];
    if (MODE_Y) {
        n_str[0] = (n_tiles + 1) >> 1;
        n_str[1] = n_tiles >> 1;
    } else {
        n_str[0] = n_tiles;
        n_str[1] = (row0 + 128 < p.B) ? n_tiles : 0;   // second row tile entirely past B: skip it
    }
    const int n_steps = n_str[0];
    // Softmax attention does not depend on the order in which KV tiles are visited.  CTAs of
    // different heads start at different tiles and wrap around, so that the CTAs resident at any
    // moment do not all read the same offset of their (power-of-two strided) per-head arrays.
    const int rot = n_tiles > 0 ? (int)(((unsigned)h * 37u + (unsigned)split * 11u) % (unsigned)n_tiles) : 0;
    auto tile_of = [&](int e) { int t = e + rot; return t_begin + (t >= n_tiles ? t - n_tiles : t); };
    // ring position of the KV tile used by stream i at step j, S buffer and its use count
    auto entry_of = [&](int j, int i) { return MODE_Y ? 2 * j + i : j; };
    auto s_col = [&](int i, int j) { return (uint32_t)(MODE_Y ? (2 * i + (j & 1)) * 64 : i * 128); };

    // Warp 0 initialises the barriers and at once issues Q and the first K and V tiles, so that the
    // first copies are in flight while the rest of the CTA sets up (tensor-memory allocation, barrier).
    const uint32_t ld0 = (warp == 0 && elect_one()) ? 1u : 0u;
    auto issue_k = [&](int e) {
        const int s = e % p.k_stages;
        uint8_t* dst = sK + s * K_TILE_BYTES;
        const int blk0 = tile_of(e) * BLK;
        mbar_arrive_expect_tx_if(ld0, &bar->k_full[s], K_TILE_BYTES);
#pragma unroll
        for (int bi = 0; bi < BLK; ++bi) {
            const int gb = h * (p.Ls_pad / 64) + blk0 + bi;
            tma_load_3d_if(ld0, dst + bi * 8192, &tm_kn, &bar->k_full[s], 0, 0, gb);
            tma_load_3d_if(ld0, dst + K_SLAB + bi * 8192, &tm_kn, &bar->k_full[s], 0, 64, gb);
            tma_load_2d_if(ld0, dst + 2 * K_SLAB + bi * 8192, &tm_kp, &bar->k_full[s], 0, (blk0 + bi) * 64);
        }
    };
    auto issue_v = [&](int e, uint32_t ld) {
        const int s = e % p.v_stages;
        const int blk0 = tile_of(e) * BLK;
        mbar_arrive_expect_tx_if(ld, &bar->v_full[s], V_TILE_BYTES);
#pragma unroll
        for (int bi = 0; bi < BLK; ++bi)
            tma_load_4d_if(ld, sV + s * V_TILE_BYTES + bi * 16384, &tm_vt, &bar->v_full[s], 0, 0, blk0 + bi, h);
    };
    if (warp == 0) {
        if (lane == 0) {
            mbar_init(&bar->q_full, 1);
            for (int s = 0; s < MAX_STAGES; ++s) {
                mbar_init(&bar->k_full[s], 1);
                mbar_init(&bar->k_empty[s], 1);
                mbar_init(&bar->v_full[s], 1);
                mbar_init(&bar->v_empty[s], 1);
            }
            for (int i = 0; i < 2; ++i) {
                for (int b = 0; b < 2; ++b) {
                    mbar_init(&bar->s_ready[i][b], 1);
                    mbar_init(&bar->p_ready[i][b], 128);
                    mbar_init(&bar->sbuf_free[i][b], 1);
                }
                mbar_init(&bar->o_done[i], 1);
            }
            bar->abort_flag = 0;
            fence_mbar_init();
        }
        __syncwarp();
        if (n_tiles > 0) {
            const int nq = (n_str[1] > 0 && !MODE_Y) ? 2 : 1;
            mbar_arrive_expect_tx_if(ld0, &bar->q_full, nq * Q_TILE_BYTES);
            for (int t = 0; t < nq; ++t) {
                uint8_t* dst = sQ + t * Q_TILE_BYTES;
                tma_load_3d_if(ld0, dst, &tm_qn, &bar->q_full, 0, h, row0 + t * 128);
                tma_load_3d_if(ld0, dst + 16384, &tm_qn, &bar->q_full, 64, h, row0 + t * 128);
                tma_load_3d_if(ld0, dst + 32768, &tm_qp, &bar->q_full, 0, h, row0 + t * 128);
            }
            // interleave K and V so that the tiles of the first steps arrive first
            for (int e = 0; e < max(p.k_stages, p.v_stages); ++e) {
                if (e < p.k_stages && e < n_tiles) issue_k(e);
                if (e < p.v_stages && e < n_tiles) issue_v(e, ld0);
            }
        }
    }
    if (warp == 1) tmem_alloc(&bar->tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // broadcast through a shuffle so that the compiler knows the value is warp-uniform
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, bar->tmem_base, 0);

    if (n_tiles > 0) {
        if (warp == 0) {
            // ---------------- K producer: the rest of the ring (Q and the first tiles are already in flight)
            for (int e = p.k_stages; e < n_tiles; ++e) {
                if (!mbar_wait_warp(&bar->k_empty[e % p.k_stages], ((e / p.k_stages) & 1) ^ 1, abort_flag)) break;
                issue_k(e);
            }
        } else if (warp == 2) {
            // ---------------- V producer
            const uint32_t ld = elect_one() ? 1u : 0u;
            for (int e = p.v_stages; e < n_tiles; ++e) {
                if (!mbar_wait_warp(&bar->v_empty[e % p.v_stages], ((e / p.v_stages) & 1) ^ 1, abort_flag)) break;
                issue_v(e, ld);
            }
        } else if (warp == 1) {
            // ---------------- S = Q K^T issuer.  With two S buffers per stream it runs ahead of the softmax
            // by up to two steps; with one it follows the PV product of the previous step.
            const uint32_t ld = elect_one() ? 1u : 0u;
            constexpr uint32_t idesc_s = idesc_bf16(128, TOK, false, false);
            bool ok = mbar_wait_warp(&bar->q_full, 0, abort_flag);
            for (int j = 0; j < n_steps && ok; ++j) {
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j >= n_str[i]) continue;
                    const int e = entry_of(j, i);
                    const int s = e % p.k_stages;
                    if (MODE_Y || i == 0) {                       // mode X: stream 1 reuses stream 0's tile
                        ok = mbar_wait_warp(&bar->k_full[s], (e / p.k_stages) & 1, abort_flag);
                        if (!ok) break;
                    }
                    if (j >= NB) {   // the PV product that read P from this S buffer NB steps ago must be done
                        ok = mbar_wait_warp(&bar->sbuf_free[i][j % NB], ((j / NB) - 1) & 1, abort_flag);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    const uint32_t qa = smem_u32(sQ + (MODE_Y ? 0 : i) * Q_TILE_BYTES);
                    const uint32_t ka = smem_u32(sK + s * K_TILE_BYTES);
                    const uint32_t d = tmem_base + s_col(i, j);
                    const bool last_user = MODE_Y || i == 1 || n_str[1] == 0;
#pragma unroll
                    for (int slab = 0; slab < 3; ++slab) {
                        const uint64_t da = smem_desc_k_sw128(qa + slab * 16384);
                        const uint64_t db = smem_desc_k_sw128(ka + slab * K_SLAB);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_ss_if(ld, d, da + 2 * k, db + 2 * k, idesc_s, (slab | k) != 0);
                    }
                    umma_commit_if(ld, &bar->s_ready[i][j % NB]);
                    if (last_user) umma_commit_if(ld, &bar->k_empty[s]);   // last user releases the ring slot
                }
            }
        } else if (warp == 3) {
            // ---------------- O += P V issuer
            const uint32_t ld = elect_one() ? 1u : 0u;
            constexpr uint32_t idesc_o = idesc_bf16(128, 128, false, false);
            bool ok = true;
            for (int j = 0; j < n_steps && ok; ++j) {
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j >= n_str[i]) continue;
                    const int e = entry_of(j, i);
                    const int s = e % p.v_stages;
                    if (MODE_Y || i == 0) {
                        ok = mbar_wait_warp(&bar->v_full[s], (e / p.v_stages) & 1, abort_flag);
                        if (!ok) break;
                    }
                    ok = mbar_wait_warp(&bar->p_ready[i][j % NB], (j / NB) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t va = smem_u32(sV + s * V_TILE_BYTES);
                    const uint32_t pa = tmem_base + s_col(i, j);
                    const uint32_t d = tmem_base + 256u + (uint32_t)i * 128u;
                    const bool last_user = MODE_Y || i == 1 || n_str[1] == 0;
#pragma unroll
                    for (int bi = 0; bi < BLK; ++bi) {
                        const uint64_t db = smem_desc_k_sw128(va + bi * 16384);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_ts_if(ld, d, pa + 8 * (bi * 4 + k), db + 2 * k, idesc_o, (j | bi | k) != 0);
                    }
                    umma_commit_if(ld, &bar->o_done[i]);
                    umma_commit_if(ld, &bar->sbuf_free[i][j % NB]);
                    if (last_user) umma_commit_if(ld, &bar->v_empty[s]);
                }
            }
        } else if (warp >= 4) {
            // ---------------- softmax warpgroups
            const int i = (warp - 4) >> 2;            // stream
            const int lg = (warp & 3) * 32;           // TMEM lane group of this warp
            const int r = lg + lane;                  // row within the 128-row tile
            const int b = row0 + (MODE_Y ? 0 : i * 128) + r;
            const int nt = n_str[i];
            const bool warp_has_rows = (b - lane) < p.B;   // warp-uniform: first row of this warp is a real request
            float m_ref = -INFINITY, l_sum = 0.f;
            bool ok = true;
            for (int j = 0; j < nt && ok; ++j) {
                const int buf = j % NB;
                ok = __all_sync(0xffffffffu, mbar_wait(&bar->s_ready[i][buf], (j / NB) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                if (!warp_has_rows) {
                    // all 32 rows of this warp are padding past B: their P rows may hold anything (rows of
                    // the MMA are independent and these output rows are never stored); just keep in step
                    tc_fence_before();
                    mbar_arrive(&bar->p_ready[i][buf]);
                    continue;
                }
                const uint32_t s_addr = tmem_base + ((uint32_t)lg << 16) + s_col(i, j);
                const int tile = tile_of(entry_of(j, i));
                const int valid = min(TOK, p.Ls - tile * TOK);
                // pass 1: row maximum of the raw logits (the scale is positive, so it commutes with the
                // maximum); the ragged tail is masked with -inf in place
                float mx_raw = -INFINITY;
                uint32_t sr[2][32];
#pragma unroll
                for (int half = 0; half < BLK; ++half) {
                    tmem_ld32(s_addr + half * 64, sr[0]);
                    tmem_ld32(s_addr + half * 64 + 32, sr[1]);
                    tmem_ld_wait();
                    if (valid < TOK) {
#pragma unroll
                        for (int c = 0; c < 64; ++c)
                            if (half * 64 + c >= valid) sr[c >> 5][c & 31] = 0xff800000u;   // -inf
                    }
#pragma unroll
                    for (int c = 0; c < 64; ++c) mx_raw = fmaxf(mx_raw, __uint_as_float(sr[c >> 5][c & 31]));
                }
                const float mx = mx_raw * p.scale_log2;
                // lazy rescale: only when some row's maximum grew by more than 2^8
                const bool grow = mx > m_ref + 8.f;
                if (j == 0) {
                    m_ref = mx;
                } else if (__any_sync(0xffffffffu, grow)) {
                    // the previous PV of this stream must have landed before O is touched
                    ok = __all_sync(0xffffffffu, mbar_wait(&bar->o_done[i], (j - 1) & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    const float m_new = grow ? mx : m_ref;
                    const float f = fast_exp2(m_ref - m_new);
                    m_ref = m_new;
                    l_sum *= f;
                    const uint32_t o_addr = tmem_base + ((uint32_t)lg << 16) + 256u + (uint32_t)i * 128u;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t orr[32];
                        tmem_ld32(o_addr + c * 32, orr);
                        tmem_ld_wait();
#pragma unroll
                        for (int q = 0; q < 32; ++q) orr[q] = __float_as_uint(__uint_as_float(orr[q]) * f);
                        tmem_st32(o_addr + c * 32, orr);
                    }
                    tmem_st_wait();
                }
                // pass 2: p = 2^(s * scale - m_ref) (one FMA and one ex2 per element), packed to bf16 over
                // the S columns (P column c holds tokens 2c, 2c+1); with 128-token tiles the logits are read
                // again, 64 at a time, to stay within the register budget
                const float neg_m = -m_ref;
#pragma unroll
                for (int half = 0; half < BLK; ++half) {
                    if (BLK == 2) {
                        tmem_ld32(s_addr + half * 64, sr[0]);
                        tmem_ld32(s_addr + half * 64 + 32, sr[1]);
                        tmem_ld_wait();
                        if (valid < TOK) {
#pragma unroll
                            for (int c = 0; c < 64; ++c)
                                if (half * 64 + c >= valid) sr[c >> 5][c & 31] = 0xff800000u;
                        }
                    }
                    uint32_t pk[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sr[(2 * c) >> 5][(2 * c) & 31]), p.scale_log2, neg_m));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sr[(2 * c + 1) >> 5][(2 * c + 1) & 31]), p.scale_log2, neg_m));
                        const uint32_t w = pack_bf16(p0, p1);
                        pk[c] = w;
                        l_sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xffff0000u);
                    }
                    // in the 128-token case the second half's logits (S columns 64-127) are loaded before
                    // P columns 32-63 are written, and P columns 0-31 only cover S columns already consumed
                    tmem_st32(s_addr + half * 32, pk);
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(&bar->p_ready[i][buf]);
            }
            // epilogue: normalised partial + LSE
            const int slot = MODE_Y ? split * 2 + i : split;
            if (nt > 0 && ok) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bar->o_done[i], (nt - 1) & 1, abort_flag));
                tc_fence_after();
            }
            if (nt > 0 && ok && warp_has_rows) {
                const float inv = 1.f / l_sum;
                const uint32_t o_addr = tmem_base + ((uint32_t)lg << 16) + 256u + (uint32_t)i * 128u;
                float* dst = p.o_part + (((int64_t)slot * p.B + b) * p.H + h) * 128;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t orr[32];
                    tmem_ld32(o_addr + c * 32, orr);
                    tmem_ld_wait();
                    if (b < p.B) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            float4 v = make_float4(__uint_as_float(orr[4 * q]) * inv, __uint_as_float(orr[4 * q + 1]) * inv,
                                                   __uint_as_float(orr[4 * q + 2]) * inv, __uint_as_float(orr[4 * q + 3]) * inv);
                            *reinterpret_cast<float4*>(dst + c * 32 + 4 * q) = v;
                        }
                    }
                }
                if (b < p.B) p.lse_part[((int64_t)slot * p.B + b) * p.H + h] = (m_ref + log2f(l_sum)) * kLn2;
            } else if (nt == 0 && b < p.B && (MODE_Y || i == 0 || row0 + 128 < p.B)) {
                p.lse_part[((int64_t)slot * p.B + b) * p.H + h] = -INFINITY;
            }
        }
    } else if (warp >= 4) {
        // empty split: every slot this CTA owns gets weight zero in the combine
        const int i = (warp - 4) >> 2;
        const int b = row0 + (MODE_Y ? 0 : i * 128) + (warp & 3) * 32 + lane;
        const int slot = MODE_Y ? split * 2 + i : split;
        if (b < p.B) p.lse_part[((int64_t)slot * p.B + b) * p.H + h] = -INFINITY;
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, 2);
        for (int k = 0; k < 64; ++k) __nanosleep(2000);   // let copies already in flight land
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace

int naive_sm100_slots(int B, int n_split) { return B <= 128 ? 2 * n_split : n_split; }
int naive_sm100_tile_tokens(int B) { return B <= 128 ? 64 : 128; }

cudaError_t launch_naive_attn_sm100(const NaiveAttnSm100& a, cudaStream_t s) {
    if (a.B <= 0 || a.Ls <= 0 || a.n_split <= 0) return cudaSuccess;
    CUtensorMap tm_qn, tm_qp;
    {
        uint64_t dims[3] = {128, (uint64_t)a.H, (uint64_t)a.B};
        uint64_t str[2] = {128 * 2, (uint64_t)a.H * 128 * 2};
        uint32_t box[3] = {64, 1, 128};
        cudaError_t e = make_tmap_bf16(&tm_qn, a.q_nope, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        uint64_t dims[3] = {64, (uint64_t)a.H, (uint64_t)a.B};
        uint64_t str[2] = {64 * 2, (uint64_t)a.H * 64 * 2};
        uint32_t box[3] = {64, 1, 128};
        cudaError_t e = make_tmap_bf16(&tm_qp, a.q_pe, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    const bool mode_y = a.B <= 128;
    NaiveSm100Params p{};
    p.B = a.B; p.H = a.H; p.Ls = a.Ls; p.Ls_pad = (a.Ls + 127) / 128 * 128;
    p.n_split = a.n_split;
    p.m_groups = mode_y ? 1 : (a.B + 255) / 256;
    p.k_stages = mode_y ? 4 : 2;
    p.v_stages = mode_y ? 4 : 1;
    p.scale_log2 = a.scale * kLog2e;
    p.o_part = a.o_part; p.lse_part = a.lse_part; p.status = a.status;
    const int k_tile = mode_y ? 64 * 384 : 128 * 384, v_tile = mode_y ? 16384 : 32768;
    const int smem = (mode_y ? 1 : 2) * Q_TILE_BYTES + p.k_stages * k_tile + p.v_stages * v_tile + 1024 + (int)sizeof(Barriers) + 64;
    dim3 grid(p.n_split * p.m_groups, a.H, 1);
    if (mode_y) {
        cudaFuncSetAttribute(naive_attn_sm100_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        naive_attn_sm100_kernel<64><<<grid, 384, smem, s>>>(tm_qn, tm_qp, *a.tm_kn, *a.tm_kp, *a.tm_vt, p);
    } else {
        cudaFuncSetAttribute(naive_attn_sm100_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        naive_attn_sm100_kernel<128><<<grid, 384, smem, s>>>(tm_qn, tm_qp, *a.tm_kn, *a.tm_kp, *a.tm_vt, p);
    }
    return cudaGetLastError();
}

cudaError_t make_naive_sm100_tmaps(const void* k_nope, const void* kpe, const void* v_t, int H, int64_t Ls_pad,
                                   CUtensorMap* tm_kn, CUtensorMap* tm_kp, CUtensorMap* tm_vt) {
    {
        // K_nope is stored as contiguous 64-token blocks of two [64 tokens][64 dims] slabs;
        // one box = one slab of one block (8 KB)
        uint64_t dims[3] = {64, 128, (uint64_t)H * (uint64_t)(Ls_pad / 64)};
        uint64_t str[2] = {64 * 2, 128 * 64 * 2};
        uint32_t box[3] = {64, 64, 1};
        cudaError_t e = make_tmap_bf16(tm_kn, k_nope, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        uint64_t dims[2] = {64, (uint64_t)Ls_pad};
        uint64_t str[1] = {64 * 2};
        uint32_t box[2] = {64, 64};
        cudaError_t e = make_tmap_bf16(tm_kp, kpe, 2, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        // V^T is stored in 64-token blocks, each a contiguous [128 dims][64 tokens] matrix
        uint64_t dims[4] = {64, 128, (uint64_t)(Ls_pad / 64), (uint64_t)H};
        uint64_t str[3] = {64 * 2, 128 * 64 * 2, (uint64_t)Ls_pad * 128 * 2};
        uint32_t box[4] = {64, 128, 1, 1};
        cudaError_t e = make_tmap_bf16(tm_vt, v_t, 4, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace tmla
