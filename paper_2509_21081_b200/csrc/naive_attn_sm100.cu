// Naive shared-prefix attention (Algorithm 1 line 4) on tcgen05 / TMEM / TMA.
//
// Per head h the step is a dense contraction over all B query rows:
//     S = Q_h [B,192] * [K_nope_h | k_pe]^T [192, L_s],  O = softmax(S) * V_h [L_s,128].
// A CTA owns one head, one group of query rows and one KV split, and runs two
// independent attention "streams" that share the TMA/MMA machinery:
//   * B > 128  (mode X): stream i = query rows [256g + 128i, +128); both streams
//     consume every 64-token KV tile of the split (tiles are loaded once).
//   * B <= 128 (mode Y): both streams use the same 128 query rows; stream i takes
//     every second KV tile (tile k -> stream k & 1) with its own softmax state, so
//     that the softmax of one stream overlaps the MMAs of the other.
// Each stream writes a normalised fp32 partial and its LSE; the combine step
// merges all partials of a (request, head).
//
// Warp roles (384 threads): warp 0 = TMA producer for Q and the K ring, warp 2 =
// TMA producer for the V ring, warp 1 = issuer of the S = Q K^T MMAs and TMEM
// owner, warp 3 = issuer of the O += P V MMAs, warps 4-7 / 8-11 = softmax
// warpgroup of stream 0 / 1 (thread = one query row).  Two issuing warps keep the
// K-side and V-side barrier waits from serialising behind each other.
//
// Tensor memory (512 columns): S[i][buf] (64 fp32 columns, P in bf16 overwrites
// the first 32) at (2i+buf)*64, O[i] (128 fp32 columns) at 256 + 128 i.
//
// Every mbarrier wait has a deadline; on expiry all roles fall through to the
// common teardown and the status word is set.
#include "kernels.h"
#include "sm100.cuh"

namespace tmla {
namespace {

using namespace sm100;

constexpr int TOK = 64;                    // tokens per KV tile
constexpr int Q_TILE_BYTES = 128 * 192 * 2;   // 3 slabs [128][64] bf16
constexpr int K_TILE_BYTES = TOK * 192 * 2;   // 3 slabs [64][64]
constexpr int V_TILE_BYTES = 128 * TOK * 2;   // [128 dims][64 tokens]
constexpr int MAX_STAGES = 4;

#ifdef TMLA_TRACE
// Debug build only: clock64 stamps of CTA (0,0): [step][slot].
__device__ long long g_trace[64 * 32];
#define TRACE(step, slot) do { if (blockIdx.x == 0 && blockIdx.y == 0 && (step) >= 0 && (step) < 64 && (threadIdx.x & 31) == 0) g_trace[(step) * 32 + (slot)] = clock64(); } while (0)
#else
#define TRACE(step, slot) do {} while (0)
#endif

struct NaiveSm100Params {
    int B, H, Ls, Ls_pad;
    int n_split, m_groups, mode_y;
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

__global__ void __launch_bounds__(384, 1)
naive_attn_sm100_kernel(const __grid_constant__ CUtensorMap tm_qn, const __grid_constant__ CUtensorMap tm_qp,
                        const __grid_constant__ CUtensorMap tm_kn, const __grid_constant__ CUtensorMap tm_kp,
                        const __grid_constant__ CUtensorMap tm_vt, NaiveSm100Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int n_q_tiles = p.mode_y ? 1 : 2;
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + n_q_tiles * Q_TILE_BYTES;
    uint8_t* sV = sK + p.k_stages * K_TILE_BYTES;
    Barriers* bar = reinterpret_cast<Barriers*>(sV + p.v_stages * V_TILE_BYTES);
    volatile int* abort_flag = &bar->abort_flag;

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    if (threadIdx.x == 0) TRACE(0, 28);
    const int split = blockIdx.x / p.m_groups, mg = blockIdx.x % p.m_groups, h = blockIdx.y;
    const int row0 = mg * (p.mode_y ? 128 : 256);

    // KV tiles of this split
    const int n_tiles_total = (p.Ls + TOK - 1) / TOK;
    const int per = (n_tiles_total + p.n_split - 1) / p.n_split;
    const int t_begin = split * per;
    const int t_end = min(n_tiles_total, t_begin + per);
    const int n_tiles = max(t_end - t_begin, 0);
    // tiles per stream and number of steps
    int n_str[2];
    if (p.mode_y) {
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

    // Warp 0 initialises the barriers and at once issues Q and the first K and V tiles, so that the
    // first copies are in flight while the rest of the CTA sets up (tensor-memory allocation, barrier).
    const uint32_t ld0 = (warp == 0 && elect_one()) ? 1u : 0u;
    auto issue_k = [&](int e) {
        const int s = e % p.k_stages;
        uint8_t* dst = sK + s * K_TILE_BYTES;
        TRACE(e >> 1, 24 + (e & 1));
        mbar_arrive_expect_tx_if(ld0, &bar->k_full[s], K_TILE_BYTES);
        tma_load_3d_if(ld0, dst, &tm_kn, &bar->k_full[s], 0, 0, h * (p.Ls_pad / TOK) + tile_of(e));
        tma_load_2d_if(ld0, dst + 16384, &tm_kp, &bar->k_full[s], 0, tile_of(e) * TOK);
    };
    auto issue_v = [&](int e, uint32_t ld) {
        const int s = e % p.v_stages;
        mbar_arrive_expect_tx_if(ld, &bar->v_full[s], V_TILE_BYTES);
        tma_load_4d_if(ld, sV + s * V_TILE_BYTES, &tm_vt, &bar->v_full[s], 0, 0, tile_of(e), h);
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
            const int nq = (n_str[1] > 0 && !p.mode_y) ? 2 : 1;
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
    if (threadIdx.x == 0) TRACE(0, 30);

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
            // ---------------- S = Q K^T issuer (whole warp runs the loop, the elected lane issues).
            // Runs ahead of the softmax by up to two steps (S is double-buffered per stream).
            const uint32_t ld = elect_one() ? 1u : 0u;
            constexpr uint32_t idesc_s = idesc_bf16(128, TOK, false, false);
            bool ok = mbar_wait_warp(&bar->q_full, 0, abort_flag);
            for (int j = 0; j < n_steps && ok; ++j) {
                TRACE(j, 0);
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j >= n_str[i]) continue;
                    const int e = p.mode_y ? 2 * j + i : j;      // ring position of this stream's KV tile
                    const int s = e % p.k_stages;
                    if (p.mode_y || i == 0) {                     // mode X: stream 1 reuses stream 0's tile
                        ok = mbar_wait_warp(&bar->k_full[s], (e / p.k_stages) & 1, abort_flag);
                        if (!ok) break;
                    }
                    if (j >= 2) {   // the PV product that read P from this S buffer two steps ago must be done
                        ok = mbar_wait_warp(&bar->sbuf_free[i][j & 1], ((j >> 1) - 1) & 1, abort_flag);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    TRACE(j, 6 + i);
                    const uint32_t qa = smem_u32(sQ + (p.mode_y ? 0 : i) * Q_TILE_BYTES);
                    const uint32_t ka = smem_u32(sK + s * K_TILE_BYTES);
                    const uint32_t d = tmem_base + (uint32_t)((2 * i + (j & 1)) * 64);
                    const bool last_user = p.mode_y || i == 1 || n_str[1] == 0;
#pragma unroll
                    for (int slab = 0; slab < 3; ++slab) {
                        const uint64_t da = smem_desc_k_sw128(qa + slab * 16384);
                        const uint64_t db = smem_desc_k_sw128(ka + slab * 8192);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_ss_if(ld, d, da + 2 * k, db + 2 * k, idesc_s, (slab | k) != 0);
                    }
                    umma_commit_if(ld, &bar->s_ready[i][j & 1]);
                    if (last_user) umma_commit_if(ld, &bar->k_empty[s]);   // last user releases the ring slot
                }
                TRACE(j, 1);
            }
        } else if (warp == 3) {
            // ---------------- O += P V issuer
            const uint32_t ld = elect_one() ? 1u : 0u;
            constexpr uint32_t idesc_o = idesc_bf16(128, 128, false, false);
            bool ok = true;
            for (int j = 0; j < n_steps && ok; ++j) {
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j >= n_str[i]) continue;
                    const int e = p.mode_y ? 2 * j + i : j;
                    const int s = e % p.v_stages;
                    if (p.mode_y || i == 0) {
                        ok = mbar_wait_warp(&bar->v_full[s], (e / p.v_stages) & 1, abort_flag);
                        if (!ok) break;
                    }
                    TRACE(j, 2 + 2 * i);
                    ok = mbar_wait_warp(&bar->p_ready[i][j & 1], (j >> 1) & 1, abort_flag);
                    if (!ok) break;
                    TRACE(j, 3 + 2 * i);
                    tc_fence_after();
                    const uint32_t va = smem_u32(sV + s * V_TILE_BYTES);
                    const uint32_t pa = tmem_base + (uint32_t)((2 * i + (j & 1)) * 64);
                    const uint32_t d = tmem_base + 256u + (uint32_t)i * 128u;
                    const uint64_t db = smem_desc_k_sw128(va);
                    const bool last_user = p.mode_y || i == 1 || n_str[1] == 0;
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_ts_if(ld, d, pa + 8 * k, db + 2 * k, idesc_o, (j | k) != 0);
                    umma_commit_if(ld, &bar->o_done[i]);
                    umma_commit_if(ld, &bar->sbuf_free[i][j & 1]);
                    if (last_user) umma_commit_if(ld, &bar->v_empty[s]);
                }
            }
        } else if (warp >= 4) {
            // ---------------- softmax warpgroups
            const int i = (warp - 4) >> 2;            // stream
            const int lg = (warp & 3) * 32;           // TMEM lane group of this warp
            const int r = lg + lane;                  // row within the 128-row tile
            const int b = row0 + (p.mode_y ? 0 : i * 128) + r;
            const int nt = n_str[i];
            const bool warp_has_rows = (b - lane) < p.B;   // warp-uniform: first row of this warp is a real request
            float m_ref = -INFINITY, l_sum = 0.f;
            bool ok = true;
            for (int j = 0; j < nt && ok; ++j) {
                const int buf = j & 1;
                if ((warp & 3) == 0 && lane == 0) TRACE(j, 8 + 8 * i);
                ok = __all_sync(0xffffffffu, mbar_wait(&bar->s_ready[i][buf], (j >> 1) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                if ((warp & 3) == 0 && lane == 0) TRACE(j, 9 + 8 * i);
                if (!warp_has_rows) {
                    // all 32 rows of this warp are padding past B: their P rows may hold anything (rows of
                    // the MMA are independent and these output rows are never stored); just keep in step
                    tc_fence_before();
                    mbar_arrive(&bar->p_ready[i][buf]);
                    continue;
                }
                const uint32_t s_addr = tmem_base + ((uint32_t)lg << 16) + (uint32_t)((2 * i + buf) * 64);
                uint32_t sr[2][32];
                tmem_ld32(s_addr, sr[0]);
                tmem_ld32(s_addr + 32, sr[1]);
                tmem_ld_wait();
                if ((warp & 3) == 0 && lane == 0) TRACE(j, 10 + 8 * i);
                // logits in base-2 units, ragged tail masked
                const int tile = tile_of(p.mode_y ? 2 * j + i : j);
                const int valid = min(TOK, p.Ls - tile * TOK);
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < 64; ++c) {
                    float v = __uint_as_float(sr[c >> 5][c & 31]) * p.scale_log2;
                    v = c < valid ? v : -INFINITY;
                    sr[c >> 5][c & 31] = __float_as_uint(v);
                    mx = fmaxf(mx, v);
                }
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
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const float p0 = fast_exp2(__uint_as_float(sr[(2 * c) >> 5][(2 * c) & 31]) - m_ref);
                    const float p1 = fast_exp2(__uint_as_float(sr[(2 * c + 1) >> 5][(2 * c + 1) & 31]) - m_ref);
                    const uint32_t w = pack_bf16(p0, p1);
                    pk[c] = w;
                    l_sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xffff0000u);
                }
                if ((warp & 3) == 0 && lane == 0) TRACE(j, 13 + 8 * i);
                tmem_st32(s_addr, pk);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(&bar->p_ready[i][buf]);
                if ((warp & 3) == 0 && lane == 0) TRACE(j, 14 + 8 * i);
            }
            // epilogue: normalised partial + LSE
            const int slot = p.mode_y ? split * 2 + i : split;
            if (nt > 0 && ok) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bar->o_done[i], (nt - 1) & 1, abort_flag));
                tc_fence_after();
            }
            if (nt > 0 && ok) {
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
            } else if (nt == 0 && b < p.B && (p.mode_y || i == 0 || row0 + 128 < p.B)) {
                p.lse_part[((int64_t)slot * p.B + b) * p.H + h] = -INFINITY;
            }
        }
    } else if (warp >= 4) {
        // empty split: every slot this CTA owns gets weight zero in the combine
        const int i = (warp - 4) >> 2;
        const int b = row0 + (p.mode_y ? 0 : i * 128) + (warp & 3) * 32 + lane;
        const int slot = p.mode_y ? split * 2 + i : split;
        if (b < p.B) p.lse_part[((int64_t)slot * p.B + b) * p.H + h] = -INFINITY;
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) TRACE(0, 29);
    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, 2);
        for (int k = 0; k < 64; ++k) __nanosleep(2000);   // let copies already in flight land
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace

#ifdef TMLA_TRACE
extern "C" int typhoon_mla_debug_read_trace(long long* dst) {
    return (int)cudaMemcpyFromSymbol(dst, g_trace, sizeof(long long) * 64 * 32);
}
#endif

int naive_sm100_slots(int B, int n_split) { return B <= 128 ? 2 * n_split : n_split; }

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
    NaiveSm100Params p{};
    p.B = a.B; p.H = a.H; p.Ls = a.Ls; p.Ls_pad = (a.Ls + 127) / 128 * 128;
    p.n_split = a.n_split;
    p.mode_y = a.B <= 128 ? 1 : 0;
    p.m_groups = p.mode_y ? 1 : (a.B + 255) / 256;
    p.k_stages = p.mode_y ? 4 : 3;
    p.v_stages = p.mode_y ? 4 : 3;
    p.scale_log2 = a.scale * kLog2e;
    p.o_part = a.o_part; p.lse_part = a.lse_part; p.status = a.status;
    const int n_q = p.mode_y ? 1 : 2;
    const int smem = n_q * Q_TILE_BYTES + p.k_stages * K_TILE_BYTES + p.v_stages * V_TILE_BYTES + 1024 + (int)sizeof(Barriers) + 64;
    cudaFuncSetAttribute(naive_attn_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    dim3 grid(p.n_split * p.m_groups, a.H, 1);
    naive_attn_sm100_kernel<<<grid, 384, smem, s>>>(tm_qn, tm_qp, *a.tm_kn, *a.tm_kp, *a.tm_vt, p);
    return cudaGetLastError();
}

cudaError_t make_naive_sm100_tmaps(const void* k_nope, const void* kpe, const void* v_t, int H, int64_t Ls_pad,
                                   CUtensorMap* tm_kn, CUtensorMap* tm_kp, CUtensorMap* tm_vt) {
    {
        // K_nope is stored as contiguous 16 KB tiles: [H * Ls_pad/64][2 slabs * 64 tokens][64 dims]
        uint64_t dims[3] = {64, 2 * TOK, (uint64_t)H * (uint64_t)(Ls_pad / TOK)};
        uint64_t str[2] = {64 * 2, 2 * TOK * 64 * 2};
        uint32_t box[3] = {64, 2 * TOK, 1};
        cudaError_t e = make_tmap_bf16(tm_kn, k_nope, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        uint64_t dims[2] = {64, (uint64_t)Ls_pad};
        uint64_t str[1] = {64 * 2};
        uint32_t box[2] = {64, TOK};
        cudaError_t e = make_tmap_bf16(tm_kp, kpe, 2, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        // V^T is stored in 64-token blocks, each a contiguous [128 dims][64 tokens] matrix
        uint64_t dims[4] = {TOK, 128, (uint64_t)(Ls_pad / TOK), (uint64_t)H};
        uint64_t str[3] = {TOK * 2, 128 * TOK * 2, (uint64_t)Ls_pad * 128 * 2};
        uint32_t box[4] = {TOK, 128, 1, 1};
        cudaError_t e = make_tmap_bf16(tm_vt, v_t, 4, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace tmla
