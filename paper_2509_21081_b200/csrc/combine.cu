// Vector kernels of the path: merge of absorb chunk partials, the final LSE
// combine (Algorithm 1 line 8; Section 3.2 "CombineLSE") and layout helpers
// used once per prefix by the expansion step.
#include <algorithm>

#include "common.cuh"
#include "kernels.h"
#include "sm100.cuh"

namespace tmla {
namespace {

// One block of G x 128 threads per (b, h) (G = 1 for a few chunks, else 4): group g takes chunks g, g+G, ...;
// each thread owns 4 of the 512 latent columns.  The chunk weights are computed once into shared
// memory, so the partial rows are fetched by independent loads (many chunks of few tokens each are
// the rule at small batch sizes, where this kernel would otherwise be a chain of dependent loads).
constexpr int MERGE_MAX_CHUNKS = 1024;
__global__ void __launch_bounds__(512) merge_latent_kernel(const float* __restrict__ o_part,
                                                           const float* __restrict__ lse_part, int n_chunks,
                                                           int BH, __nv_bfloat16* __restrict__ o_lat,
                                                           float* __restrict__ lse) {
    sm100::pdl_trigger();
    sm100::pdl_wait();
    __shared__ float w_s[MERGE_MAX_CHUNKS];
    __shared__ float red[16];
    __shared__ float4 acc_s[3][128];
    const int bh = blockIdx.x, tid = threadIdx.x, grp = tid >> 7, col = tid & 127;
    const int nthr = blockDim.x, G = nthr >> 7, nwarp = nthr >> 5;
    // maximum of the chunk LSEs
    float m = -INFINITY;
    for (int c = tid; c < n_chunks; c += nthr) {
        const float l = lse_part[(int64_t)c * BH + bh];
        w_s[c] = l;
        m = fmaxf(m, l);
    }
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((tid & 31) == 0) red[tid >> 5] = m;
    __syncthreads();
    m = red[0];
    for (int i = 1; i < nwarp; ++i) m = fmaxf(m, red[i]);
    __syncthreads();
    // weights (0 for an empty chunk, whose O slot was never written) and their sum
    float z = 0.f;
    for (int c = tid; c < n_chunks; c += nthr) {
        const float l = w_s[c];
        const float w = (l == -INFINITY) ? 0.f : __expf(l - m);
        w_s[c] = w;
        z += w;
    }
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if ((tid & 31) == 0) red[tid >> 5] = z;
    __syncthreads();
    z = 0.f;
    for (int i = 0; i < nwarp; ++i) z += red[i];
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (m != -INFINITY) {
        const float* src = o_part + (int64_t)bh * 512 + col * 4;
        // loads do not wait for the weights (eight in flight per thread); an empty chunk's slot was never
        // written, so its value is dropped by a select
#pragma unroll 8
        for (int c = grp; c < n_chunks; c += G) {
            const float4 v = *reinterpret_cast<const float4*>(src + (int64_t)c * BH * 512);
            const float w = w_s[c];
            const bool live = w != 0.f;
            acc.x += live ? w * v.x : 0.f; acc.y += live ? w * v.y : 0.f;
            acc.z += live ? w * v.z : 0.f; acc.w += live ? w * v.w : 0.f;
        }
    }
    if (grp > 0) acc_s[grp - 1][col] = acc;
    __syncthreads();
    if (grp == 0) {
        for (int g = 0; g < G - 1; ++g) {
            const float4 v = acc_s[g][col];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        if (m != -INFINITY) {
            const float inv = 1.f / z;
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        }
        uint2 pk = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
        *reinterpret_cast<uint2*>(o_lat + (int64_t)bh * 512 + col * 4) = pk;
        if (col == 0) lse[bh] = (m == -INFINITY) ? -INFINITY : m + __logf(z);
    }
}

// Few chunks per request (the common case at larger batch sizes): no shared memory, four (b, h) rows
// per block of 512 threads, each thread owns 4 of a row's 512 latent columns and recomputes the (at most
// NC) chunk weights itself.  The LSEs and the partial rows are all requested before any of them is used
// (one memory round trip per thread); the slot of an empty chunk was never written, so its value is
// dropped by a select, not multiplied by a zero weight.
constexpr int MERGE_FEW = 16;
template <int NC>
__global__ void __launch_bounds__(512) merge_latent_few_kernel(const float* __restrict__ o_part,
                                                               const float* __restrict__ lse_part, int n_chunks,
                                                               int BH, __nv_bfloat16* __restrict__ o_lat,
                                                               float* __restrict__ lse) {
    sm100::pdl_trigger();
    sm100::pdl_wait();
    const int bh = blockIdx.x * 4 + (threadIdx.x >> 7), col = threadIdx.x & 127;
    if (bh >= BH) return;
    float l[NC];
    float4 v[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) l[c] = c < n_chunks ? lse_part[(int64_t)c * BH + bh] : -INFINITY;
#pragma unroll
    for (int c = 0; c < NC; ++c)
        v[c] = c < n_chunks ? *reinterpret_cast<const float4*>(o_part + ((int64_t)c * BH + bh) * 512 + col * 4)
                            : make_float4(0.f, 0.f, 0.f, 0.f);
    float m = -INFINITY;
#pragma unroll
    for (int c = 0; c < NC; ++c) m = fmaxf(m, l[c]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float z = 0.f;
    if (m != -INFINITY) {
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const bool live = l[c] != -INFINITY;
            const float w = live ? __expf(l[c] - m) : 0.f;
            acc.x += live ? w * v[c].x : 0.f; acc.y += live ? w * v[c].y : 0.f;
            acc.z += live ? w * v[c].z : 0.f; acc.w += live ? w * v[c].w : 0.f;
            z += w;
        }
        const float inv = 1.f / z;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    uint2 pk = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
    *reinterpret_cast<uint2*>(o_lat + (int64_t)bh * 512 + col * 4) = pk;
    if (col == 0) lse[bh] = (m == -INFINITY) ? -INFINITY : m + __logf(z);
}

// Absorb-only step at small batch sizes: merge of the chunk partials, output projection O_A W_UV^T (Algorithm 1
// line 7) and the final rounding in one launch.  One block per (request, head), 512 threads.  The 128 KB of the
// head's W_UV (16 warps x 8 rows x 1 KB) are requested into L2 first and arrive while the chunk partials are merged
// as in merge_latent_kernel; the merged latent row stays in fp32 in shared memory; every warp then forms 8 of the 128
// outputs as dot products over 512 (16 elements per lane, butterfly sum).  Each block re-reads its head's weights,
// so this form is for one or two requests (the GEMM form reads them once per 128 requests).
__global__ void __launch_bounds__(512) merge_project_kernel(const float* __restrict__ o_part,
                                                            const float* __restrict__ lse_part, int n_chunks, int B,
                                                            int H, const __nv_bfloat16* __restrict__ w_uv,
                                                            void* __restrict__ out, float* __restrict__ lse_out,
                                                            int out_fp32) {
    sm100::pdl_trigger();
    sm100::pdl_wait();
    __shared__ float w_s[MERGE_MAX_CHUNKS];
    __shared__ float red[16];
    __shared__ float4 acc_s[4][128];
    const int h = blockIdx.x, b = blockIdx.y, BH = B * H, bh = b * H + h;
    const int tid = threadIdx.x, grp = tid >> 7, col = tid & 127, warp = tid >> 5, lane = tid & 31;
    // this warp's 8 weight rows (8 KB, contiguous): requested into L2 now, loaded after the merge
    const __nv_bfloat16* wrow = w_uv + ((int64_t)h * 128 + warp * 8) * 512 + lane * 16;
    {
        const char* wl = reinterpret_cast<const char*>(w_uv + ((int64_t)h * 128 + warp * 8) * 512);
        asm volatile("prefetch.global.L2 [%0];\n" ::"l"(wl + lane * 128));
        asm volatile("prefetch.global.L2 [%0];\n" ::"l"(wl + 4096 + lane * 128));
    }
    float m = -INFINITY;
    for (int c = tid; c < n_chunks; c += 512) {
        const float l = lse_part[(int64_t)c * BH + bh];
        w_s[c] = l;
        m = fmaxf(m, l);
    }
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[warp] = m;
    __syncthreads();
    m = red[0];
    for (int i = 1; i < 16; ++i) m = fmaxf(m, red[i]);
    __syncthreads();
    float z = 0.f;
    for (int c = tid; c < n_chunks; c += 512) {
        const float l = w_s[c];
        const float w = (l == -INFINITY) ? 0.f : __expf(l - m);
        w_s[c] = w;
        z += w;
    }
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if (lane == 0) red[warp] = z;
    __syncthreads();
    z = 0.f;
    for (int i = 0; i < 16; ++i) z += red[i];
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (m != -INFINITY) {
        const float* src = o_part + (int64_t)bh * 512 + col * 4;
#pragma unroll 4
        for (int c = grp; c < n_chunks; c += 4) {
            const float4 v = *reinterpret_cast<const float4*>(src + (int64_t)c * BH * 512);
            const float w = w_s[c];
            const bool live = w != 0.f;   // an empty chunk's slot was never written
            acc.x += live ? w * v.x : 0.f; acc.y += live ? w * v.y : 0.f;
            acc.z += live ? w * v.z : 0.f; acc.w += live ? w * v.w : 0.f;
        }
    }
    acc_s[grp][col] = acc;
    __syncthreads();
    // the merged, normalised latent row: this lane's 16 elements (float4 columns 4 lane .. 4 lane + 3)
    const float inv = (m != -INFINITY) ? 1.f / z : 0.f;
    float o[16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float4 v = acc_s[0][lane * 4 + q];
#pragma unroll
        for (int g = 1; g < 4; ++g) {
            const float4 u = acc_s[g][lane * 4 + q];
            v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
        }
        o[4 * q] = v.x * inv; o[4 * q + 1] = v.y * inv; o[4 * q + 2] = v.z * inv; o[4 * q + 3] = v.w * inv;
    }
    uint4 wv[8][2];   // 16 consecutive elements per lane and row (two 16-byte loads)
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        wv[r][0] = *reinterpret_cast<const uint4*>(wrow + r * 512);
        wv[r][1] = *reinterpret_cast<const uint4*>(wrow + r * 512 + 8);
    }
    float res = 0.f;   // lane r < 8 keeps output row warp * 8 + r
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const uint32_t wr[8] = {wv[r][0].x, wv[r][0].y, wv[r][0].z, wv[r][0].w, wv[r][1].x, wv[r][1].y, wv[r][1].z, wv[r][1].w};
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const __nv_bfloat162 p2 = *reinterpret_cast<const __nv_bfloat162*>(&wr[e]);
            d += __low2float(p2) * o[2 * e] + __high2float(p2) * o[2 * e + 1];
        }
        for (int s2 = 16; s2 > 0; s2 >>= 1) d += __shfl_xor_sync(0xffffffffu, d, s2);
        if (lane == r) res = d;
    }
    if (lane < 8) {
        const int64_t idx = (int64_t)bh * 128 + warp * 8 + lane;
        if (out_fp32) reinterpret_cast<float*>(out)[idx] = res;
        else reinterpret_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(res);
    }
    if (tid == 0 && lse_out != nullptr) lse_out[bh] = (m == -INFINITY) ? -INFINITY : m + __logf(z);
}

// One warp per (b, h); each lane owns 4 of the 128 output columns.
__global__ void __launch_bounds__(256) combine_kernel(const float* __restrict__ o_naive,
                                                      const float* __restrict__ lse_naive, int n_naive,
                                                      const float* __restrict__ o_abs,
                                                      const float* __restrict__ lse_abs, int BH,
                                                      void* __restrict__ out, float* __restrict__ lse_out, int out_fp32) {
    sm100::pdl_trigger();
    sm100::pdl_wait();
    const int bh = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (bh >= BH) return;
    float m = -INFINITY;
    for (int i = 0; i < n_naive; ++i) m = fmaxf(m, lse_naive[(int64_t)i * BH + bh]);
    float la = -INFINITY;
    if (o_abs != nullptr) {
        la = lse_abs[bh];
        m = fmaxf(m, la);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float z = 0.f;
    if (m != -INFINITY) {
        for (int i = 0; i < n_naive; ++i) {
            float l = lse_naive[(int64_t)i * BH + bh];
            if (l == -INFINITY) continue;
            float w = __expf(l - m);
            float4 v = *reinterpret_cast<const float4*>(o_naive + ((int64_t)i * BH + bh) * 128 + lane * 4);
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
            z += w;
        }
        if (la != -INFINITY) {
            float w = __expf(la - m);
            float4 v = *reinterpret_cast<const float4*>(o_abs + (int64_t)bh * 128 + lane * 4);
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
            z += w;
        }
        float inv = 1.f / z;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    if (out_fp32) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + (int64_t)bh * 128 + lane * 4) = acc;
    } else {
        uint2 pk = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + (int64_t)bh * 128 + lane * 4) = pk;
    }
    if (lse_out != nullptr && lane == 0) lse_out[bh] = (m == -INFINITY) ? -INFINITY : m + __logf(z);
}

__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16* __restrict__ in,
                                                             __nv_bfloat16* __restrict__ out, int R, int C) {
    __shared__ __nv_bfloat16 tile[32][34];
    const int64_t off = (int64_t)blockIdx.z * R * C;
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        int r = r0 + i, c = c0 + tx;
        tile[i][tx] = (r < R && c < C) ? in[off + (int64_t)r * C + c] : __float2bfloat16(0.f);
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        int c = c0 + i, r = r0 + tx;
        if (r < R && c < C) out[off + (int64_t)c * R + r] = tile[tx][i];
    }
}

__global__ void __launch_bounds__(256) copy_pad_rows_kernel(const __nv_bfloat16* __restrict__ in, int64_t ld_in,
                                                            __nv_bfloat16* __restrict__ out, int L, int Lp, int W8) {
    int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    int64_t total = (int64_t)Lp * W8;
    if (idx >= total) return;
    int row = (int)(idx / W8), ch = (int)(idx % W8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < L) v = *reinterpret_cast<const uint4*>(in + (int64_t)row * ld_in + ch * 8);
    *reinterpret_cast<uint4*>(out + ((int64_t)row * W8 + ch) * 8) = v;
}

// Longest-first launch order for ragged suffixes: perm[] = request indices sorted by descending
// suffix length (ties by index, so the order is deterministic).  One block, bitonic sort in
// shared memory of up to 4096 keys.
__global__ void __launch_bounds__(1024) order_by_length_kernel(const int32_t* __restrict__ seq_lens, int B,
                                                               int32_t* __restrict__ perm) {
    __shared__ unsigned long long keys[4096];
    block_order_by_length(seq_lens, B, perm, keys);
}

// -inf into n_slots segments of `count` floats, `stride` floats apart (LSE of partial slots no kernel fills).
__global__ void __launch_bounds__(256) fill_neg_inf_kernel(float* __restrict__ dst, int n_slots, int64_t stride, int64_t count) {
    const int64_t total = (int64_t)n_slots * count;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256)
        dst[(i / count) * stride + i % count] = -INFINITY;
}

// Row expansion for S_q query tokens per request (Table 1's S_q; causal among the new tokens):
// row b * S_q + j gets request b's page-table row and the suffix length minus the S_q - 1 - j later tokens.
__global__ void __launch_bounds__(256) expand_query_rows_kernel(const int32_t* __restrict__ block_table,
                                                                const int32_t* __restrict__ seq_lens, int B,
                                                                int max_pages, int S_q,
                                                                int32_t* __restrict__ bt_rows,
                                                                int32_t* __restrict__ len_rows) {
    const int64_t n_bt = (int64_t)B * S_q * max_pages;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n_bt; i += (int64_t)gridDim.x * 256) {
        const int64_t row = i / max_pages;
        bt_rows[i] = block_table[(row / S_q) * max_pages + i % max_pages];
    }
    for (int i = blockIdx.x * 256 + threadIdx.x; i < B * S_q; i += gridDim.x * 256)
        len_rows[i] = max(seq_lens[i / S_q] - (S_q - 1 - i % S_q), 0);
}

}  // namespace

// Test kernel for the bounded wait of the tcgen05 kernels: a barrier on which nothing arrives, the same
// mbar_wait with a short deadline, the same report through the status word, a normal return.
static __global__ void wait_expiry_selftest_kernel(int* status, long long deadline_cycles, int code) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        sm100::mbar_init(&bar, 1);
        abort_flag = 0;
        sm100::fence_mbar_init();
    }
    __syncthreads();
    const bool ok = sm100::mbar_wait(&bar, 0, &abort_flag, deadline_cycles);   // nobody arrives: runs out
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_flag) && status) atomicOr(status, code);
}
cudaError_t launch_wait_expiry_selftest(int* status, long long deadline_cycles, int code, cudaStream_t s) {
    wait_expiry_selftest_kernel<<<1, 32, 0, s>>>(status, deadline_cycles, code);
    return cudaGetLastError();
}

cudaError_t launch_order_by_length(const int32_t* seq_lens, int B, int32_t* perm, cudaStream_t s) {
    if (B <= 0 || B > 4096) return cudaErrorInvalidValue;
    order_by_length_kernel<<<1, 1024, 0, s>>>(seq_lens, B, perm);
    return cudaGetLastError();
}

cudaError_t launch_fill_neg_inf(float* dst, int n_slots, int64_t stride, int64_t count, cudaStream_t s) {
    if (n_slots <= 0 || count <= 0) return cudaSuccess;
    const int64_t total = (int64_t)n_slots * count;
    fill_neg_inf_kernel<<<(unsigned)std::min<int64_t>((total + 255) / 256, 1184), 256, 0, s>>>(dst, n_slots, stride, count);
    return cudaGetLastError();
}

cudaError_t launch_expand_query_rows(const int32_t* block_table, const int32_t* seq_lens, int B, int max_pages, int S_q,
                                     int32_t* bt_rows, int32_t* len_rows, cudaStream_t s) {
    if (B <= 0 || S_q <= 0) return cudaSuccess;
    const int64_t n = std::max<int64_t>((int64_t)B * S_q * max_pages, (int64_t)B * S_q);
    const unsigned blocks = (unsigned)std::min<int64_t>((n + 255) / 256, 1184);
    expand_query_rows_kernel<<<blocks, 256, 0, s>>>(block_table, seq_lens, B, max_pages, S_q, bt_rows, len_rows);
    return cudaGetLastError();
}

cudaError_t launch_merge_project(const float* o_part, const float* lse_part, int n_chunks, int B, int H, const void* w_uv,
                                 void* out, float* lse_out, bool out_fp32, cudaStream_t s) {
    if (B * H <= 0) return cudaSuccess;
    if (n_chunks > MERGE_MAX_CHUNKS) return cudaErrorInvalidValue;
    return launch_pdl(merge_project_kernel, dim3(H, B), dim3(512), 0, s, o_part, lse_part, n_chunks, B, H,
                      reinterpret_cast<const __nv_bfloat16*>(w_uv), out, lse_out, out_fp32 ? 1 : 0);
}

cudaError_t launch_merge_latent(const float* o_part, const float* lse_part, int n_chunks, int B, int H,
                                void* o_lat_bf16, float* lse, cudaStream_t s) {
    if (B * H <= 0) return cudaSuccess;
    if (n_chunks > MERGE_MAX_CHUNKS) return cudaErrorInvalidValue;
    if (n_chunks <= MERGE_FEW) {
        const dim3 grid((B * H + 3) / 4);
        __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(o_lat_bf16);
        if (n_chunks <= 2) return launch_pdl(merge_latent_few_kernel<2>, grid, dim3(512), 0, s, o_part, lse_part, n_chunks, B * H, o, lse);
        if (n_chunks <= 4) return launch_pdl(merge_latent_few_kernel<4>, grid, dim3(512), 0, s, o_part, lse_part, n_chunks, B * H, o, lse);
        if (n_chunks <= 8) return launch_pdl(merge_latent_few_kernel<8>, grid, dim3(512), 0, s, o_part, lse_part, n_chunks, B * H, o, lse);
        return launch_pdl(merge_latent_few_kernel<MERGE_FEW>, grid, dim3(512), 0, s, o_part, lse_part, n_chunks, B * H, o, lse);
    } else {
        return launch_pdl(merge_latent_kernel, dim3(B * H), dim3(512), 0, s, o_part, lse_part, n_chunks, B * H,
                          reinterpret_cast<__nv_bfloat16*>(o_lat_bf16), lse);
    }
    return cudaGetLastError();
}

cudaError_t launch_combine(const float* o_naive, const float* lse_naive, int n_naive, const float* o_abs,
                           const float* lse_abs, int B, int H, void* out, float* lse_out, cudaStream_t s, bool out_fp32) {
    int BH = B * H;
    if (BH <= 0) return cudaSuccess;
    return launch_pdl(combine_kernel, dim3((BH + 7) / 8), dim3(256), 0, s, o_naive, lse_naive, n_naive, o_abs, lse_abs, BH,
                      out, lse_out, out_fp32 ? 1 : 0);
}

cudaError_t launch_transpose_bf16(const void* in, void* out, int R, int C, int batch, cudaStream_t s) {
    if (R <= 0 || C <= 0 || batch <= 0) return cudaSuccess;
    dim3 grid((C + 31) / 32, (R + 31) / 32, batch);
    transpose_bf16_kernel<<<grid, 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(in),
                                               reinterpret_cast<__nv_bfloat16*>(out), R, C);
    return cudaGetLastError();
}

cudaError_t launch_copy_pad_rows(const void* in, int64_t ld_in, void* out, int L, int Lp, int W, cudaStream_t s) {
    if (Lp <= 0) return cudaSuccess;
    int W8 = W / 8;
    int64_t total = (int64_t)Lp * W8;
    copy_pad_rows_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
        reinterpret_cast<const __nv_bfloat16*>(in), ld_in, reinterpret_cast<__nv_bfloat16*>(out), L, Lp, W8);
    return cudaGetLastError();
}

}  // namespace tmla
