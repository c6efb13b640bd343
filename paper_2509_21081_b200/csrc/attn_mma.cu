// Warp-MMA (mma.sync) attention kernels: the portable-path implementation of
//   * the naive shared-prefix attention (Algorithm 1 line 4), and
//   * the absorb attention over latent tokens (Algorithm 1 line 6),
// each producing normalised fp32 partials plus natural-log LSEs per KV split,
// to be merged by the combine step (Algorithm 1 line 8).
//
// Both are flash-decoding style: a CTA owns a tile of query rows and a range
// of KV tokens, streams KV tiles through shared memory with cp.async, and keeps
// an online softmax (running max / sum in base 2) in registers.
#include "common.cuh"
#include "kernels.h"

namespace tmla {
namespace {

// Shared-memory addressing: rows of CH 16-byte chunks; the low three bits of
// the chunk index are XOR-ed with the row so that 8 consecutive rows of one
// logical chunk fall in 8 distinct 16-byte bank groups (ldmatrix conflict-free).
template <int CH>
__device__ __forceinline__ int swz(int row, int chunk) {
    return (row * CH + ((chunk & ~7) | ((chunk ^ row) & 7))) << 3;
}

// ---------------------------------------------------------------------------
// Naive shared-prefix attention.  grid = (n_split, ceil(B/64), H), 128 threads.
// Rows of the tile are requests b (one head h per CTA); K = [K_nope | k_pe]
// (192 wide), V^T tile is [128 dims][64 tokens].
// ---------------------------------------------------------------------------
constexpr int NA_ROWS = 64, NA_TOK = 64;
constexpr int NA_Q_ELEMS = NA_ROWS * 192;
constexpr int NA_K_ELEMS = NA_TOK * 192;
constexpr int NA_V_ELEMS = 128 * NA_TOK;
constexpr int NA_STAGE_ELEMS = NA_K_ELEMS + NA_V_ELEMS;
constexpr int NA_SMEM_BYTES = (NA_Q_ELEMS + 2 * NA_STAGE_ELEMS) * 2;

__global__ void __launch_bounds__(128) naive_attn_mma_kernel(NaiveAttn p) {
    extern __shared__ __align__(128) __nv_bfloat16 smem[];
    __nv_bfloat16* sQ = smem;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, b0 = blockIdx.y * NA_ROWS, h = blockIdx.z;
    const int n_tiles = (p.Ls + NA_TOK - 1) / NA_TOK;
    const int per = (n_tiles + p.n_split - 1) / p.n_split;
    const int t_begin = split * per, t_end = min(n_tiles, t_begin + per);

    const __nv_bfloat16* qn = reinterpret_cast<const __nv_bfloat16*>(p.q_nope);
    const __nv_bfloat16* qp = reinterpret_cast<const __nv_bfloat16*>(p.q_pe);
    const __nv_bfloat16* kn = reinterpret_cast<const __nv_bfloat16*>(p.k_nope) + (int64_t)h * p.Ls_pad * 128;
    const __nv_bfloat16* vt = reinterpret_cast<const __nv_bfloat16*>(p.v_t) + (int64_t)h * 128 * p.Ls_pad;  // [Lp/64][128][64]
    const __nv_bfloat16* kr = reinterpret_cast<const __nv_bfloat16*>(p.kpe);

    const int r_lo = lane >> 2;  // this thread's rows within the warp's 16: r_lo and r_lo + 8

    if (t_begin >= t_end) {  // empty split: weight zero in the combine
        for (int i = tid; i < NA_ROWS; i += 128) {
            int b = b0 + i;
            if (b < p.B) p.lse_part[((int64_t)split * p.B + b) * p.H + h] = -INFINITY;
        }
        return;
    }

    // Q tile -> smem (rows >= B zero-filled)
    for (int idx = tid; idx < NA_ROWS * 24; idx += 128) {
        int row = idx / 24, ch = idx % 24;
        int b = b0 + row;
        bool ok = b < p.B;
        int bb = ok ? b : 0;
        const __nv_bfloat16* src = ch < 16 ? qn + ((int64_t)bb * p.H + h) * 128 + ch * 8
                                           : qp + ((int64_t)bb * p.H + h) * 64 + (ch - 16) * 8;
        cp_async16(smem_u32(sQ + swz<24>(row, ch)), src, ok);
    }
    cp_async_commit();

    auto load_tile = [&](int stage, int tile) {
        __nv_bfloat16* sK = smem + NA_Q_ELEMS + stage * NA_STAGE_ELEMS;
        __nv_bfloat16* sV = sK + NA_K_ELEMS;
        const int t0 = tile * NA_TOK;
        for (int idx = tid; idx < NA_TOK * 24; idx += 128) {
            int row = idx / 24, ch = idx % 24;
            const __nv_bfloat16* src = ch < 16 ? kn + (((int64_t)tile * 2 + (ch >> 3)) << 12) + (row << 6) + (ch & 7) * 8
                                               : kr + (int64_t)(t0 + row) * 64 + (ch - 16) * 8;
            cp_async16(smem_u32(sK + swz<24>(row, ch)), src, true);
        }
        for (int idx = tid; idx < 128 * 8; idx += 128) {
            int row = idx >> 3, ch = idx & 7;
            cp_async16(smem_u32(sV + swz<8>(row, ch)), vt + ((int64_t)tile * 128 + row) * 64 + ch * 8, true);
        }
    };

    load_tile(0, t_begin);
    cp_async_commit();

    // Q fragments to registers
    cp_async_wait<1>();
    __syncthreads();
    uint32_t qf[12][4];
#pragma unroll
    for (int ks = 0; ks < 12; ++ks)
        ldmatrix_x4(qf[ks], smem_u32(sQ + swz<24>(warp * 16 + (lane & 15), ks * 2 + (lane >> 4))));

    float o[16][4];
#pragma unroll
    for (int j = 0; j < 16; ++j)
#pragma unroll
        for (int k = 0; k < 4; ++k) o[j][k] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const float sl2 = p.scale * kLog2e;

    for (int tile = t_begin; tile < t_end; ++tile) {
        const int stage = (tile - t_begin) & 1;
        if (tile + 1 < t_end) load_tile(stage ^ 1, tile + 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const __nv_bfloat16* sK = smem + NA_Q_ELEMS + stage * NA_STAGE_ELEMS;
        const __nv_bfloat16* sV = sK + NA_K_ELEMS;

        float s[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k) s[j][k] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 12; ++ks) {
#pragma unroll
            for (int jp = 0; jp < 4; ++jp) {
                uint32_t bfr[4];
                int row = jp * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldmatrix_x4(bfr, smem_u32(sK + swz<24>(row, ks * 2 + ((lane >> 3) & 1))));
                mma_bf16(s[jp * 2], qf[ks], bfr[0], bfr[1]);
                mma_bf16(s[jp * 2 + 1], qf[ks], bfr[2], bfr[3]);
            }
        }
        // scale, mask the ragged tail, tile max
        const int t0 = tile * NA_TOK;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                int tok = t0 + j * 8 + (lane & 3) * 2 + (k & 1);
                float v = tok < p.Ls ? s[j][k] * sl2 : -INFINITY;
                s[j][k] = v;
                mx[k >> 1] = fmaxf(mx[k >> 1], v);
            }
        float corr[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            float m_new = fmaxf(m_run[r], mx[r]);  // finite: every tile holds at least one valid token
            corr[r] = fast_exp2(m_run[r] - m_new);
            m_run[r] = m_new;
            l_run[r] *= corr[r];
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            o[j][0] *= corr[0]; o[j][1] *= corr[0];
            o[j][2] *= corr[1]; o[j][3] *= corr[1];
        }
        uint32_t pf[4][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float e0 = bf16_round(fast_exp2(s[j][0] - m_run[0]));
            float e1 = bf16_round(fast_exp2(s[j][1] - m_run[0]));
            float e2 = bf16_round(fast_exp2(s[j][2] - m_run[1]));
            float e3 = bf16_round(fast_exp2(s[j][3] - m_run[1]));
            l_run[0] += e0 + e1;
            l_run[1] += e2 + e3;
            pf[j >> 1][(j & 1) * 2] = pack_bf16(e0, e1);
            pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(e2, e3);
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int jp = 0; jp < 8; ++jp) {
                uint32_t bfr[4];
                int row = jp * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldmatrix_x4(bfr, smem_u32(sV + swz<8>(row, kk * 2 + ((lane >> 3) & 1))));
                mma_bf16(o[jp * 2], pf[kk], bfr[0], bfr[1]);
                mma_bf16(o[jp * 2 + 1], pf[kk], bfr[2], bfr[3]);
            }
        }
        __syncthreads();
    }
    cp_async_wait<0>();

#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        int b = b0 + warp * 16 + r_lo + r * 8;
        if (b >= p.B) continue;
        float inv = 1.f / l_run[r];
        int64_t base = ((int64_t)split * p.B + b) * p.H + h;
        float* dst = p.o_part + base * 128;
#pragma unroll
        for (int j = 0; j < 16; ++j)
            *reinterpret_cast<float2*>(dst + j * 8 + (lane & 3) * 2) = make_float2(o[j][r * 2] * inv, o[j][r * 2 + 1] * inv);
        if ((lane & 3) == 0) p.lse_part[base] = (m_run[r] + log2f(l_run[r])) * kLn2;
    }
}

// ---------------------------------------------------------------------------
// Absorb attention over latent tokens.  grid = (n_chunks, H/64 (ceil), B),
// 256 threads: warps 0-3 / 4-7 own latent columns 0-255 / 256-511 of the
// output for the same four 16-row groups of heads.  The KV tile is
// [32 tokens][576] = [latent 512 | rope 64]; the latent part doubles as V.
// ---------------------------------------------------------------------------
constexpr int AB_ROWS = 64, AB_TOK = 32;
constexpr int AB_Q_ELEMS = AB_ROWS * 576;
constexpr int AB_KV_ELEMS = AB_TOK * 576;
constexpr int AB_SMEM_BYTES = (AB_Q_ELEMS + 2 * AB_KV_ELEMS) * 2;

__global__ void __launch_bounds__(256) absorb_attn_mma_kernel(AbsorbAttn p) {
    extern __shared__ __align__(128) __nv_bfloat16 smem[];
    __nv_bfloat16* sQ = smem;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = warp & 3, chalf = warp >> 2;
    const int chunk = blockIdx.x, h0 = blockIdx.y * AB_ROWS;
    const int b = p.order ? p.order[blockIdx.z] : (int)blockIdx.z;
    const int n_chunks = p.n_shared_chunks + p.n_suffix_chunks;

    // token range of this chunk
    const bool shared_seg = chunk < p.n_shared_chunks;
    int seg_len, tok_begin;
    if (shared_seg) {
        seg_len = p.Ls_absorb;
        tok_begin = chunk * p.chunk;
    } else {
        int cap = p.max_pages * p.page_size;
        seg_len = min(max(p.seq_lens[b], 0), cap);
        tok_begin = (chunk - p.n_shared_chunks) * p.chunk;
    }
    const int tok_end = min(seg_len, tok_begin + p.chunk);
    (void)n_chunks;

    if (tok_begin >= tok_end) {
        for (int i = tid; i < AB_ROWS; i += 256) {
            int h = h0 + i;
            if (h < p.H) p.lse_part[((int64_t)chunk * p.B + b) * p.H + h] = -INFINITY;
        }
        return;
    }

    const __nv_bfloat16* qa = reinterpret_cast<const __nv_bfloat16*>(p.q_abs);
    const __nv_bfloat16* qp = reinterpret_cast<const __nv_bfloat16*>(p.q_pe);
    for (int idx = tid; idx < AB_ROWS * 72; idx += 256) {
        int row = idx / 72, ch = idx % 72;
        int h = h0 + row;
        bool ok = h < p.H;
        int hh = ok ? h : 0;
        const __nv_bfloat16* src = ch < 64 ? qa + ((int64_t)b * p.H + hh) * 512 + ch * 8
                                           : qp + ((int64_t)b * p.H + hh) * 64 + (ch - 64) * 8;
        cp_async16(smem_u32(sQ + swz<72>(row, ch)), src, ok);
    }
    cp_async_commit();

    const __nv_bfloat16* ckv_s = reinterpret_cast<const __nv_bfloat16*>(p.ckv_shared);
    const __nv_bfloat16* kpe_s = reinterpret_cast<const __nv_bfloat16*>(p.kpe_shared);
    const __nv_bfloat16* ckv_p = reinterpret_cast<const __nv_bfloat16*>(p.ckv_pages);
    const __nv_bfloat16* kpe_p = reinterpret_cast<const __nv_bfloat16*>(p.kpe_pages);
    const int32_t* bt = p.block_table + (int64_t)b * p.max_pages;

    auto load_tile = [&](int stage, int t0) {
        __nv_bfloat16* sKV = smem + AB_Q_ELEMS + stage * AB_KV_ELEMS;
        for (int idx = tid; idx < AB_TOK * 72; idx += 256) {
            int row = idx / 72, ch = idx % 72;
            int tok = t0 + row;
            bool ok = tok < tok_end;
            const __nv_bfloat16* src;
            if (shared_seg) {
                int t = ok ? tok : 0;
                src = ch < 64 ? ckv_s + (int64_t)t * 512 + ch * 8 : kpe_s + (int64_t)t * 64 + (ch - 64) * 8;
            } else {
                int t = ok ? tok : tok_begin;
                int pg = bt[t / p.page_size];
                if ((unsigned)pg >= (unsigned)p.num_pages) {   // not dereferenced: the token reads as zeros
                    if (ok && p.status) atomicOr(p.status, 0x100);
                    ok = false;
                    pg = 0;
                }
                int64_t slot = (int64_t)pg * p.page_size + (t % p.page_size);
                src = ch < 64 ? ckv_p + slot * p.ckv_stride + ch * 8 : kpe_p + slot * p.kpe_stride + (ch - 64) * 8;
            }
            cp_async16(smem_u32(sKV + swz<72>(row, ch)), src, ok);
        }
    };

    load_tile(0, tok_begin);
    cp_async_commit();

    float o[32][4];
#pragma unroll
    for (int j = 0; j < 32; ++j)
#pragma unroll
        for (int k = 0; k < 4; ++k) o[j][k] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const float sl2 = p.scale * kLog2e;
    const int n_tiles = (tok_end - tok_begin + AB_TOK - 1) / AB_TOK;

    for (int it = 0; it < n_tiles; ++it) {
        const int stage = it & 1;
        const int t0 = tok_begin + it * AB_TOK;
        if (it + 1 < n_tiles) load_tile(stage ^ 1, t0 + AB_TOK);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const __nv_bfloat16* sKV = smem + AB_Q_ELEMS + stage * AB_KV_ELEMS;

        float s[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k) s[j][k] = 0.f;
#pragma unroll 4
        for (int ks = 0; ks < 36; ++ks) {
            uint32_t a[4];
            ldmatrix_x4(a, smem_u32(sQ + swz<72>(rg * 16 + (lane & 15), ks * 2 + (lane >> 4))));
#pragma unroll
            for (int jp = 0; jp < 2; ++jp) {
                uint32_t bfr[4];
                int row = jp * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldmatrix_x4(bfr, smem_u32(sKV + swz<72>(row, ks * 2 + ((lane >> 3) & 1))));
                mma_bf16(s[jp * 2], a, bfr[0], bfr[1]);
                mma_bf16(s[jp * 2 + 1], a, bfr[2], bfr[3]);
            }
        }
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                int tok = t0 + j * 8 + (lane & 3) * 2 + (k & 1);
                float v = tok < tok_end ? s[j][k] * sl2 : -INFINITY;
                s[j][k] = v;
                mx[k >> 1] = fmaxf(mx[k >> 1], v);
            }
        float corr[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            float m_new = fmaxf(m_run[r], mx[r]);
            corr[r] = fast_exp2(m_run[r] - m_new);
            m_run[r] = m_new;
            l_run[r] *= corr[r];
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            o[j][0] *= corr[0]; o[j][1] *= corr[0];
            o[j][2] *= corr[1]; o[j][3] *= corr[1];
        }
        uint32_t pf[2][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float e0 = bf16_round(fast_exp2(s[j][0] - m_run[0]));
            float e1 = bf16_round(fast_exp2(s[j][1] - m_run[0]));
            float e2 = bf16_round(fast_exp2(s[j][2] - m_run[1]));
            float e3 = bf16_round(fast_exp2(s[j][3] - m_run[1]));
            l_run[0] += e0 + e1;
            l_run[1] += e2 + e3;
            pf[j >> 1][(j & 1) * 2] = pack_bf16(e0, e1);
            pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(e2, e3);
        }
        // O[16][256] += P[16][32] * C[32][256 of this warp's half]
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
            for (int jp = 0; jp < 16; ++jp) {
                uint32_t bfr[4];
                int row = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                int ch = chalf * 32 + jp * 2 + (lane >> 4);
                ldmatrix_x4_trans(bfr, smem_u32(sKV + swz<72>(row, ch)));
                mma_bf16(o[jp * 2], pf[kk], bfr[0], bfr[1]);
                mma_bf16(o[jp * 2 + 1], pf[kk], bfr[2], bfr[3]);
            }
        }
        __syncthreads();
    }
    cp_async_wait<0>();

#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        int h = h0 + rg * 16 + (lane >> 2) + r * 8;
        if (h >= p.H) continue;
        float inv = 1.f / l_run[r];
        int64_t base = ((int64_t)chunk * p.B + b) * p.H + h;
        float* dst = p.o_part + base * 512 + chalf * 256;
#pragma unroll
        for (int j = 0; j < 32; ++j)
            *reinterpret_cast<float2*>(dst + j * 8 + (lane & 3) * 2) = make_float2(o[j][r * 2] * inv, o[j][r * 2 + 1] * inv);
        if (chalf == 0 && (lane & 3) == 0) p.lse_part[base] = (m_run[r] + log2f(l_run[r])) * kLn2;
    }
}

}  // namespace

cudaError_t set_attrs_attn_mma() {
    cudaError_t e = cudaFuncSetAttribute(naive_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, NA_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(absorb_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AB_SMEM_BYTES);
    return e;
}

cudaError_t launch_naive_attn_mma(const NaiveAttn& p, cudaStream_t s) {
    if (p.B <= 0 || p.Ls <= 0 || p.n_split <= 0) return cudaSuccess;
    dim3 grid(p.n_split, (p.B + NA_ROWS - 1) / NA_ROWS, p.H);
    naive_attn_mma_kernel<<<grid, 128, NA_SMEM_BYTES, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_absorb_attn_mma(const AbsorbAttn& p, cudaStream_t s) {
    int n_chunks = p.n_shared_chunks + p.n_suffix_chunks;
    if (p.B <= 0 || n_chunks <= 0) return cudaSuccess;
    dim3 grid(n_chunks, (p.H + AB_ROWS - 1) / AB_ROWS, p.B);
    absorb_attn_mma_kernel<<<grid, 256, AB_SMEM_BYTES, s>>>(p);
    return cudaGetLastError();
}

}  // namespace tmla
